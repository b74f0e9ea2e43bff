// libthc: kernels and C ABI.  See include/thc.h for the contract of every entry point.
//
// Structure of the transform.  An RHT block of B = 2^k coordinates with k <= 14 is handled by
// rht_tile_kernel below: a CTA holds a tile of 2^14 consecutive coordinates (one block or
// several small ones) in shared memory: load (+ sign flip or de-quantisation), stages of
// stride 1 .. 2^(k-1), then the fused epilogue: scale by 1/sqrt(B) and either truncate +
// quantise + pack (compress), sign flip + store (decompress) or min / max (exact range).
// Larger blocks go through the persistent two-pass pipeline of thc_pipeline.cuh.
#include "../../include/thc.h"
#include "thc_device.cuh"

#include <math.h>
#include <mutex>
#include <new>
#include <stdio.h>
#include <string.h>

namespace thc {

struct PtrArray { const void *p[THC_MAX_WORKERS]; };
struct MutPtrArray { void *p[THC_MAX_WORKERS]; };

enum LoadKind { kLoadGradF32, kLoadGradBF16, kLoadSum8, kLoadSum16, kLoadSum32 };
enum StoreKind { kStoreQuant, kStoreOut, kStoreRange };

// Geometry of the tiles one launch walks.
struct TileGeom {
    uint64_t d;            // valid coordinates per worker
    uint64_t d_pad;
    uint64_t row_stride;   // coordinates between consecutive tile rows
    uint32_t k;            // log2 of the RHT block
    uint32_t row_log2;     // tile = 2^row_log2 rows ...
    uint32_t col_log2;     // ... of 2^col_log2 consecutive coordinates (sum = 14)
    uint32_t lo_cbit;      // chunk-index bits [lo_cbit, hi_cbit) are transformed
    uint32_t hi_cbit;
    uint32_t blocks_in_tile;   // RHT blocks a tile overlaps (1 if k >= 14)
    uint32_t lut_rep;          // lane replication of the quantiser table in shared memory
    uint32_t granularity;
    uint32_t divisor;          // decompress: workers summed
    uint32_t round;
    uint32_t worker_base;
    float    c_block;          // (float)(1/sqrt(B))
    uint32_t exact_range;      // scales = nblocks minima then nblocks maxima (else M per block)
};

__device__ __forceinline__ uint64_t tile_base(const TileGeom &g, uint32_t tile)
{
    if (g.row_log2 == 0) return (uint64_t)tile << kTileLog2;
    const uint32_t panels = 1u << g.row_log2;          // panels per RHT block
    const uint64_t blk = tile >> g.row_log2;
    const uint64_t panel = tile & (panels - 1);
    return (blk << g.k) + (panel << g.col_log2);
}

__device__ __forceinline__ uint64_t chunk_coord(const TileGeom &g, uint64_t base, int c)
{
    const int ccl = (int)g.col_log2 - 2;
    const uint64_t row = (uint64_t)(c >> ccl);
    const uint64_t cc = (uint64_t)(c & ((1 << ccl) - 1));
    return base + row * g.row_stride + cc * 4;
}

// Sign words of every row of the tile, 32 coordinates per word.
__device__ __forceinline__ void fill_sign_words(uint32_t *sw, const TileGeom &g, uint64_t base,
                                                const PhiloxKeys &keys, int tid,
                                                int nthreads = kThreads)
{
    const int cols = 1 << g.col_log2;
    const int words_per_row = max(1, cols >> 5);
    const int calls_per_row = max(1, cols >> 7);
    const int rows = 1 << g.row_log2;
    const int words_per_call = min(4, words_per_row);
    for (int q = tid; q < rows * calls_per_row; q += nthreads) {
        const int row = q / calls_per_row;
        const int cr = q - row * calls_per_row;
        const uint64_t j0 = base + (uint64_t)row * g.row_stride + (uint64_t)cr * 128;
        const uint4 ph = sign_call(j0, g.round, keys);
        const int first = (int)((j0 >> 5) & 3);
        for (int wi = 0; wi < words_per_call; ++wi) {
            const int src = first + wi;
            const uint32_t w = src == 0 ? ph.x : src == 1 ? ph.y : src == 2 ? ph.z : ph.w;
            sw[row * words_per_row + cr * 4 + wi] = w;
        }
    }
}

__device__ __forceinline__ uint32_t sign_bits_of_chunk(const uint32_t *sw, const TileGeom &g,
                                                       int c, uint64_t j)
{
    const int ccl = (int)g.col_log2 - 2;
    const int row = c >> ccl;
    const int cc = c & ((1 << ccl) - 1);
    const int words_per_row = max(1, (1 << g.col_log2) >> 5);
    return sw[row * words_per_row + (cc >> 3)] >> (uint32_t)(j & 31);
}

__device__ __forceinline__ float4 load_f32x4_masked(const float *x, uint64_t j, uint64_t d)
{
    if (j + 4 <= d) return __ldg(reinterpret_cast<const float4 *>(x + j));
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (j + 0 < d) v.x = __ldg(x + j + 0);
    if (j + 1 < d) v.y = __ldg(x + j + 1);
    if (j + 2 < d) v.z = __ldg(x + j + 2);
    if (j + 3 < d) v.w = __ldg(x + j + 3);
    return v;
}

// Eight 3-bit indices (24 bits, coordinate 0 in the low bits) go to bytes 3 (j/8) .. +2.
__device__ __forceinline__ void store_packed3(unsigned char *pk, uint64_t j, uint32_t z)
{
    unsigned char *p = pk + 3 * (j >> 3);
    p[0] = (unsigned char)z;
    p[1] = (unsigned char)(z >> 8);
    p[2] = (unsigned char)(z >> 16);
}

__device__ __forceinline__ float sum_to_float(uint32_t y)   // exact for y < 2^23
{
    return __uint_as_float(0x4B000000u | y) - 8388608.0f;
}

// One tile: load, butterfly rounds, store.  blockIdx.x = tile, blockIdx.y = local worker.
template <int LOAD, int STORE, int BITS, bool IDENTITY>
__global__ void __launch_bounds__(kThreads, 2)
rht_tile_kernel(TileGeom g, PtrArray in, MutPtrArray out, MutPtrArray rotated,
                const float *__restrict__ scales, DeviceBlock *dev, PhiloxKeys keys)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float4 *tile = reinterpret_cast<float4 *>(smem_raw);
    uint32_t *sw = reinterpret_cast<uint32_t *>(smem_raw + kTileElems * 4);
    float2 *blk_const = reinterpret_cast<float2 *>(smem_raw + kTileElems * 4 + kSignWordsMax * 4);
    unsigned char *lut = smem_raw + kTileElems * 4 + kSignWordsMax * 4 +
                         (((size_t)g.blocks_in_tile * 8 + 15) & ~(size_t)15);

    const int tid = threadIdx.x;
    const uint32_t wl = blockIdx.y;
    const uint64_t base = tile_base(g, blockIdx.x);
    const uint64_t first_blk = base >> g.k;
    const uint64_t nblocks = g.d_pad >> g.k;

    // ---- per-tile constants
    if (LOAD == kLoadGradF32 || LOAD == kLoadGradBF16 || STORE == kStoreOut)
        fill_sign_words(sw, g, base, keys, tid);
    if (STORE == kStoreQuant) {
        // (1/(2M), 1/2) per block; (0, 0) for a degenerate block
        for (uint32_t b = tid; b < g.blocks_in_tile; b += kThreads) {
            float2 c = make_float2(0.f, 0.f);
            if (first_blk + b < nblocks)
                c = compress_constants(block_range(scales, first_blk + b, nblocks, g.exact_range));
            blk_const[b] = c;
        }
        if (!IDENTITY) lut_fill<LutKind<BITS, IDENTITY>::k8>(lut, dev, g.granularity, tid, kThreads);
    }
    if (LOAD == kLoadSum8 || LOAD == kLoadSum16 || LOAD == kLoadSum32) {
        // (step, -M) per block; (0, 0) for a degenerate block
        for (uint32_t b = tid; b < g.blocks_in_tile; b += kThreads) {
            float2 c = make_float2(0.f, 0.f);
            if (first_blk + b < nblocks)
                c = decode_constants(block_range(scales, first_blk + b, nblocks, g.exact_range),
                                     g.granularity, g.divisor);
            blk_const[b] = c;
        }
    }
    __syncthreads();

    // ---- load phase
    if (LOAD == kLoadGradF32) {
        const float *x = static_cast<const float *>(in.p[wl]);
#pragma unroll 4
        for (int i = 0; i < kTileChunks / kThreads; ++i) {
            const int c = tid + i * kThreads;
            const uint64_t j = base + (uint64_t)c * 4;
            float4 v = load_f32x4_masked(x, j, g.d);
            v = flip4(v, sw[c >> 3] >> ((c & 7) * 4));
            tile[swz(c)] = stages01(v);
        }
    } else if (LOAD == kLoadGradBF16) {
        const uint16_t *x = static_cast<const uint16_t *>(in.p[wl]);
#pragma unroll 2
        for (int i = 0; i < kTileChunks / 2 / kThreads; ++i) {
            const int u = tid + i * kThreads;                 // 8 coordinates
            const uint64_t j = base + (uint64_t)u * 8;
            uint32_t w[4] = {0, 0, 0, 0};
            if (j + 8 <= g.d) {
                const uint4 q = __ldg(reinterpret_cast<const uint4 *>(x + j));
                w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w;
            } else {
                for (int e = 0; e < 8; ++e)
                    if (j + e < g.d) w[e >> 1] |= (uint32_t)__ldg(x + j + e) << ((e & 1) * 16);
            }
            float4 v0 = make_float4(__uint_as_float(w[0] << 16), __uint_as_float(w[0] & 0xFFFF0000u),
                                    __uint_as_float(w[1] << 16), __uint_as_float(w[1] & 0xFFFF0000u));
            float4 v1 = make_float4(__uint_as_float(w[2] << 16), __uint_as_float(w[2] & 0xFFFF0000u),
                                    __uint_as_float(w[3] << 16), __uint_as_float(w[3] & 0xFFFF0000u));
            const int c = 2 * u;
            const uint32_t bits = sw[c >> 3] >> ((c & 7) * 4);
            tile[swz(c)] = stages01(flip4(v0, bits));
            tile[swz(c + 1)] = stages01(flip4(v1, bits >> 4));
        }
    } else if (LOAD == kLoadSum8 || LOAD == kLoadSum16 || LOAD == kLoadSum32) {
        constexpr int kPer = LOAD == kLoadSum8 ? 16 : LOAD == kLoadSum16 ? 8 : 4;   // sums per 16 B
        const unsigned char *y = static_cast<const unsigned char *>(in.p[0]);
        for (int i = 0; i < kTileElems / kPer / kThreads; ++i) {
            const int u = tid + i * kThreads;
            const uint64_t j = base + (uint64_t)u * kPer;
            uint4 q = make_uint4(0, 0, 0, 0);
            if (j + kPer <= g.d_pad) {
                q = __ldg(reinterpret_cast<const uint4 *>(y + j * (16 / kPer)));
            } else if (j < g.d_pad) {          // only 8-bit sums with 8-coordinate blocks
                const uint2 h = __ldg(reinterpret_cast<const uint2 *>(y + j * (16 / kPer)));
                q.x = h.x; q.y = h.y;
            }
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int cc = 0; cc < kPer / 4; ++cc) {
                uint64_t bi = ((j + cc * 4) >> g.k) - first_blk;
                if (bi >= g.blocks_in_tile) bi = 0;
                const float2 bc = blk_const[bi];
                float s[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int idx = cc * 4 + e;
                    uint32_t val;
                    if (LOAD == kLoadSum8) val = (w[idx >> 2] >> ((idx & 3) * 8)) & 0xFFu;
                    else if (LOAD == kLoadSum16) val = (w[idx >> 1] >> ((idx & 1) * 16)) & 0xFFFFu;
                    else val = w[idx];
                    const float yf = LOAD == kLoadSum32 ? (float)val : sum_to_float(val);
                    s[e] = fmaf(yf, bc.x, bc.y);
                }
                tile[swz(u * (kPer / 4) + cc)] = stages01(make_float4(s[0], s[1], s[2], s[3]));
            }
        }
    }
    __syncthreads();

    // ---- butterflies
    fwht_rounds(tile, (int)g.lo_cbit, (int)g.hi_cbit, tid);

    // ---- store phase
    if (STORE == kStoreQuant) {
        unsigned char *pk = static_cast<unsigned char *>(out.p[wl]);
        float *rot = static_cast<float *>(rotated.p[wl]);
        const float gf = (float)g.granularity;
        const uint32_t my_lut = lut_lane_addr<LutKind<BITS, IDENTITY>::k8>(lut, tid);
#pragma unroll 1
        for (int i = 0; i < kTileChunks / 2 / kThreads; ++i) {
            const int u = tid + i * kThreads;
            const int c = 2 * u;
            const uint64_t j = chunk_coord(g, base, c);
            if (j >= g.d_pad) continue;
            const float4 a = scale4(tile[swz(c)], g.c_block);
            const float4 b = scale4(tile[swz(c + 1)], g.c_block);
            if (rot != nullptr) {
                *reinterpret_cast<float4 *>(rot + j) = a;
                *reinterpret_cast<float4 *>(rot + j + 4) = b;
            }
            const float r[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
            const float2 bc = blk_const[(j >> g.k) - first_blk];
            const uint4 rnd = round_call(j, g.worker_base + wl, g.round, keys);
            const uint64_t z = quantize8<BITS, IDENTITY>(r, bc.x, bc.y, gf, rnd, my_lut);
            if constexpr (BITS == 8) *reinterpret_cast<uint2 *>(pk + j) = make_uint2((uint32_t)z, (uint32_t)(z >> 32));
            else if constexpr (BITS == 4) *reinterpret_cast<uint32_t *>(pk + j / 2) = (uint32_t)z;
            else if constexpr (BITS == 3) store_packed3(pk, j, (uint32_t)z);
            else if constexpr (BITS == 2) *reinterpret_cast<uint16_t *>(pk + j / 4) = (uint16_t)z;
            else pk[j / 8] = (unsigned char)z;
        }
    } else if (STORE == kStoreRange) {
        // min / max of the rotated coordinates per RHT block, as ordered keys: out.p[0] holds
        // nblocks min keys followed by nblocks max keys.  For blocks of at least 128
        // coordinates the 32 chunks of a warp lie in one block and are reduced first.
        uint32_t *rk = static_cast<uint32_t *>(out.p[0]);
#pragma unroll 1
        for (int i = 0; i < kTileChunks / kThreads; ++i) {
            const int c = tid + i * kThreads;
            const uint64_t j = chunk_coord(g, base, c);
            if (j >= g.d_pad) continue;
            const float4 v = scale4(tile[swz(c)], g.c_block);
            if (rotated.p[wl] != nullptr) *reinterpret_cast<float4 *>(static_cast<float *>(rotated.p[wl]) + j) = v;
            const uint32_t k0 = float_key(v.x), k1 = float_key(v.y), k2 = float_key(v.z), k3 = float_key(v.w);
            uint32_t kmin = min(min(k0, k1), min(k2, k3));
            uint32_t kmax = max(max(k0, k1), max(k2, k3));
            const uint64_t blk = j >> g.k;
            if (g.k >= 7) {
                kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
                kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
                if ((tid & 31) != 0) continue;
            }
            atomicMin(rk + blk, kmin);
            atomicMax(rk + nblocks + blk, kmax);
        }
    } else {   // kStoreOut
        float *o = static_cast<float *>(out.p[0]);
#pragma unroll 4
        for (int i = 0; i < kTileChunks / kThreads; ++i) {
            const int c = tid + i * kThreads;
            const uint64_t j = chunk_coord(g, base, c);
            if (j >= g.d) continue;
            float4 v = scale4(tile[swz(c)], g.c_block);
            v = flip4(v, sign_bits_of_chunk(sw, g, c, j));
            if (j + 4 <= g.d) {
                *reinterpret_cast<float4 *>(o + j) = v;
            } else {
                o[j] = v.x;
                if (j + 1 < g.d) o[j + 1] = v.y;
                if (j + 2 < g.d) o[j + 2] = v.z;
            }
        }
    }
}

constexpr int kQrBlockCache = 1024;

// Quantise + pack coordinates that are already rotated (the epilogue of compress alone).
template <int BITS, bool IDENTITY>
__global__ void __launch_bounds__(kThreads)
quantize_rotated_kernel(PtrArray rotated, MutPtrArray packed, uint64_t d_pad, uint32_t k,
                        uint32_t granularity, uint32_t round, uint32_t worker_base, uint32_t exact_range,
                        const float *__restrict__ scales, const DeviceBlock *dev, PhiloxKeys keys)
{
    // dynamic shared memory: the quantiser table, one copy per lane group, then the block
    // constants of the first kQrBlockCache RHT blocks (the fp64 division is done once per block)
    extern __shared__ __align__(16) unsigned char qr_smem[];
    unsigned char *lut = qr_smem;
    float2 *bc = reinterpret_cast<float2 *>(qr_smem + (size_t)(granularity + 1) * kLutEntryBytes);
    if (!IDENTITY) lut_fill<LutKind<BITS, IDENTITY>::k8>(lut, dev, granularity, threadIdx.x, kThreads);
    const uint64_t nblocks = d_pad >> k;
    const uint32_t cached = nblocks < (uint64_t)kQrBlockCache ? (uint32_t)nblocks : (uint32_t)kQrBlockCache;
    for (uint32_t b = threadIdx.x; b < cached; b += kThreads)
        bc[b] = compress_constants(block_range(scales, b, nblocks, exact_range));
    __syncthreads();
    const uint32_t wl = blockIdx.y;
    const float *rot = static_cast<const float *>(rotated.p[wl]);
    unsigned char *pk = static_cast<unsigned char *>(packed.p[wl]);
    const float gf = (float)granularity;
    const uint32_t my_lut = lut_lane_addr<LutKind<BITS, IDENTITY>::k8>(lut, threadIdx.x);
    for (uint64_t u = (uint64_t)blockIdx.x * kThreads + threadIdx.x; u < d_pad / 8;
         u += (uint64_t)gridDim.x * kThreads) {
        const uint64_t j = u * 8;
        const float4 a = __ldg(reinterpret_cast<const float4 *>(rot + j));
        const float4 b = __ldg(reinterpret_cast<const float4 *>(rot + j + 4));
        const float r[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        const uint64_t blk = j >> k;
        const float2 kc = blk < cached ? bc[blk] : compress_constants(block_range(scales, blk, nblocks, exact_range));
        const float kappa = kc.x, offset = kc.y;
        const uint4 rnd = round_call(j, worker_base + wl, round, keys);
        const uint64_t z = quantize8<BITS, IDENTITY>(r, kappa, offset, gf, rnd, my_lut);
        if constexpr (BITS == 8) *reinterpret_cast<uint2 *>(pk + j) = make_uint2((uint32_t)z, (uint32_t)(z >> 32));
        else if constexpr (BITS == 4) *reinterpret_cast<uint32_t *>(pk + j / 2) = (uint32_t)z;
        else if constexpr (BITS == 3) store_packed3(pk, j, (uint32_t)z);
        else if constexpr (BITS == 2) *reinterpret_cast<uint16_t *>(pk + j / 4) = (uint16_t)z;
        else pk[j / 8] = (unsigned char)z;
    }
}

// Fast path of the PS sum for 4-bit indices, 8-bit sums and table values below 128 (the
// paper's prototype: 4-bit indices, 8-bit table values and sums, Section 3).  The 16 table
// bytes sit in four registers; `prmt` looks four indices up at once.  A selector nibble with
// bit 3 set makes prmt return the sign of the selected byte, i.e. 0 for values < 128, so the
// low half of the table answers indices 0-7 and, with bit 3 flipped, the high half answers
// 8-15; the two results are disjoint and are added into packed byte accumulators (no byte
// can overflow because workers * g <= 255).
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

__global__ void __launch_bounds__(kThreads)
aggregate_b4w8_kernel(PtrArray in, uint32_t n, uint64_t units32, const DeviceBlock *dev,
                      uint4 *__restrict__ sum)
{
    uint32_t t[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
        t[q] = dev->table[4 * q] | (dev->table[4 * q + 1] << 8) | (dev->table[4 * q + 2] << 16) |
               (dev->table[4 * q + 3] << 24);
    // A thread sums 32 coordinates: 16 bytes of indices per worker, the loads of up to eight
    // workers in flight together, 32 bytes of sums out.
    for (uint64_t u = (uint64_t)blockIdx.x * kThreads + threadIdx.x; u < units32;
         u += (uint64_t)gridDim.x * kThreads) {
        uint32_t acc[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};     // 32 sums of 8 bits
#pragma unroll 1
        for (uint32_t i0 = 0; i0 < n; i0 += 8) {
            uint4 w[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)         // index 0 everywhere adds T[0] = 0
                w[j] = i0 + j < n ? __ldcs(reinterpret_cast<const uint4 *>(in.p[i0 + j]) + u) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t words[4] = {w[j].x, w[j].y, w[j].z, w[j].w};
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const uint32_t a = words[h], b = a ^ 0x88888888u;
                    acc[2 * h] += prmt(t[0], t[1], a) + prmt(t[2], t[3], b);
                    acc[2 * h + 1] += prmt(t[0], t[1], a >> 16) + prmt(t[2], t[3], b >> 16);
                }
            }
        }
        __stcs(sum + 2 * u, make_uint4(acc[0], acc[1], acc[2], acc[3]));
        __stcs(sum + 2 * u + 1, make_uint4(acc[4], acc[5], acc[6], acc[7]));
    }
}

// The same with 16-bit sums (more workers than fit a byte: workers * g > 255).  Table values are
// summed in byte lanes for CHUNK workers at a time (CHUNK * g <= 255), then widened into
// 16-bit lanes (even and odd coordinates apart) and put back in order at the end.
template <int CHUNK>
__global__ void __launch_bounds__(kThreads)
aggregate_b4w16_kernel(PtrArray in, uint32_t n, uint64_t units32, const DeviceBlock *dev,
                       uint4 *__restrict__ sum)
{
    uint32_t t[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
        t[q] = dev->table[4 * q] | (dev->table[4 * q + 1] << 8) | (dev->table[4 * q + 2] << 16) |
               (dev->table[4 * q + 3] << 24);
    // A thread sums 32 coordinates: 16 bytes of indices per worker, 64 bytes of sums out.
    for (uint64_t u = (uint64_t)blockIdx.x * kThreads + threadIdx.x; u < units32;
         u += (uint64_t)gridDim.x * kThreads) {
        uint32_t even[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u}, odd[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll 1
        for (uint32_t i0 = 0; i0 < n; i0 += CHUNK) {
            uint4 w[CHUNK];
#pragma unroll
            for (int j = 0; j < CHUNK; ++j)      // index 0 everywhere adds T[0] = 0
                w[j] = i0 + j < n ? __ldcs(reinterpret_cast<const uint4 *>(in.p[i0 + j]) + u) : make_uint4(0u, 0u, 0u, 0u);
            uint32_t acc[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
            for (int j = 0; j < CHUNK; ++j) {
                const uint32_t words[4] = {w[j].x, w[j].y, w[j].z, w[j].w};
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const uint32_t a = words[h], b = a ^ 0x88888888u;
                    acc[2 * h] += prmt(t[0], t[1], a) + prmt(t[2], t[3], b);
                    acc[2 * h + 1] += prmt(t[0], t[1], a >> 16) + prmt(t[2], t[3], b >> 16);
                }
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                even[q] += acc[q] & 0x00FF00FFu;
                odd[q] += (acc[q] >> 8) & 0x00FF00FFu;
            }
        }
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t o[4];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                o[2 * q] = prmt(even[2 * q4 + q], odd[2 * q4 + q], 0x5410u);          // coordinates 4q, 4q+1
                o[2 * q + 1] = prmt(even[2 * q4 + q], odd[2 * q4 + q], 0x7632u);      // coordinates 4q+2, 4q+3
            }
            __stcs(sum + 4 * u + q4, make_uint4(o[0], o[1], o[2], o[3]));
        }
    }
}

// 1- and 2-bit indices with 8-bit sums: T[z] = g z for one bit, the identity table for two, so
// the sum of table values is g times the sum of the indices.  Index fields are spread into
// byte lanes by shift and mask (lane j of the k-th spread holds coordinate (8/BITS) j + k), added
// across workers, and transposed into coordinate order at the end.  A thread handles 32
// coordinates.
template <int BITS>
__global__ void __launch_bounds__(kThreads)
aggregate_small_w8_kernel(PtrArray in, uint32_t n, uint64_t units32, uint32_t g_mult,
                          uint4 *__restrict__ sum)
{
    constexpr int kWords = BITS;                       // 32 coordinates = BITS words
    constexpr int kSpread = 8 / BITS;                  // spreads per word
    constexpr uint32_t kMask = BITS == 1 ? 0x01010101u : 0x03030303u;
    for (uint64_t u = (uint64_t)blockIdx.x * kThreads + threadIdx.x; u < units32;
         u += (uint64_t)gridDim.x * kThreads) {
        uint32_t acc[kWords][kSpread];
#pragma unroll
        for (int q = 0; q < kWords; ++q)
#pragma unroll
            for (int k = 0; k < kSpread; ++k) acc[q][k] = 0u;
#pragma unroll 4
        for (uint32_t i = 0; i < n; ++i) {
            uint32_t words[kWords];
            if constexpr (BITS == 1) {
                words[0] = __ldg(reinterpret_cast<const uint32_t *>(in.p[i]) + u);
            } else {
                const uint2 w = __ldg(reinterpret_cast<const uint2 *>(in.p[i]) + u);
                words[0] = w.x; words[1] = w.y;
            }
#pragma unroll
            for (int q = 0; q < kWords; ++q)
#pragma unroll
                for (int k = 0; k < kSpread; ++k) acc[q][k] += (words[q] >> (k * BITS)) & kMask;
        }
        // byte j of acc[q][k] is coordinate (32/BITS) q + kSpread j + k: gather four consecutive
        // coordinates into each output word
        uint32_t o[8];
#pragma unroll
        for (int q = 0; q < kWords; ++q) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int h = 0; h < kSpread / 4; ++h) {
                    const uint32_t *a = &acc[q][4 * h];
                    const uint32_t sel = (uint32_t)j | ((uint32_t)(4 + j) << 4);
                    const uint32_t p01 = prmt(a[0], a[1], sel);            // bytes: a0[j], a1[j]
                    const uint32_t p23 = prmt(a[2], a[3], sel);            // bytes: a2[j], a3[j]
                    const uint32_t word = prmt(p01, p23, 0x5410u);         // a0[j], a1[j], a2[j], a3[j]
                    o[(q * (32 / BITS) + kSpread * j + 4 * h) / 4] = word * g_mult;
                }
            }
        }
        sum[2 * u] = make_uint4(o[0], o[1], o[2], o[3]);
        sum[2 * u + 1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

// 8-bit indices with the identity table (g = 255) and 16-bit sums: bytes are widened into
// 16-bit lanes (even and odd coordinates apart).  A thread handles 16 coordinates.
__global__ void __launch_bounds__(kThreads)
aggregate_b8w16_kernel(PtrArray in, uint32_t n, uint64_t units16, uint4 *__restrict__ sum)
{
    for (uint64_t u = (uint64_t)blockIdx.x * kThreads + threadIdx.x; u < units16;
         u += (uint64_t)gridDim.x * kThreads) {
        uint32_t even[4] = {0u, 0u, 0u, 0u}, odd[4] = {0u, 0u, 0u, 0u};
#pragma unroll 4
        for (uint32_t i = 0; i < n; ++i) {
            const uint4 w = __ldg(reinterpret_cast<const uint4 *>(in.p[i]) + u);
            const uint32_t words[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                even[q] += words[q] & 0x00FF00FFu;
                odd[q] += (words[q] >> 8) & 0x00FF00FFu;
            }
        }
        uint32_t o[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            o[2 * q] = prmt(even[q], odd[q], 0x5410u);
            o[2 * q + 1] = prmt(even[q], odd[q], 0x7632u);
        }
        sum[2 * u] = make_uint4(o[0], o[1], o[2], o[3]);
        sum[2 * u + 1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

// ------------------------------------------------------------------------ error feedback
// e <- x - e (e holds RHT^-1(X) on entry) and x <- x + e, 128-bit accesses with a scalar tail.
__global__ void __launch_bounds__(kThreads)
ef_subtract_kernel(const float *__restrict__ x, float *__restrict__ e, uint64_t d)
{
    const uint64_t n4 = d / 4;
    for (uint64_t c = (uint64_t)blockIdx.x * kThreads + threadIdx.x; c < n4; c += (uint64_t)gridDim.x * kThreads) {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(x) + c);
        float4 b = reinterpret_cast<float4 *>(e)[c];
        b.x = a.x - b.x; b.y = a.y - b.y; b.z = a.z - b.z; b.w = a.w - b.w;
        reinterpret_cast<float4 *>(e)[c] = b;
    }
    if (blockIdx.x == 0 && threadIdx.x < (d & 3)) {
        const uint64_t j = n4 * 4 + threadIdx.x;
        e[j] = x[j] - e[j];
    }
}

__global__ void __launch_bounds__(kThreads)
accumulate_kernel(float *__restrict__ x, const float *__restrict__ e, uint64_t d)
{
    const uint64_t n4 = d / 4;
    for (uint64_t c = (uint64_t)blockIdx.x * kThreads + threadIdx.x; c < n4; c += (uint64_t)gridDim.x * kThreads) {
        float4 a = reinterpret_cast<float4 *>(x)[c];
        const float4 b = __ldg(reinterpret_cast<const float4 *>(e) + c);
        a.x = a.x + b.x; a.y = a.y + b.y; a.z = a.z + b.z; a.w = a.w + b.w;
        reinterpret_cast<float4 *>(x)[c] = a;
    }
    if (blockIdx.x == 0 && threadIdx.x < (d & 3)) {
        const uint64_t j = n4 * 4 + threadIdx.x;
        x[j] = x[j] + e[j];
    }
}

// ------------------------------------------------------------------------------ prepare
// Partial sums of squares in fp64: one CTA per (chunk of 2^chunk_log2 coordinates, worker).
template <bool BF16>
__global__ void __launch_bounds__(kThreads)
prepare_partial_kernel(PtrArray in, uint64_t d, uint32_t chunk_log2, uint64_t chunks_per_worker,
                       double *__restrict__ partial)
{
    const uint64_t chunk = blockIdx.x;
    const uint32_t wl = blockIdx.y;
    const uint64_t j0 = chunk << chunk_log2;
    const int n4 = 1 << (chunk_log2 - 2);
    double s = 0.0;
    if (BF16) {
        // eight bf16 (16 bytes) per load
        const uint16_t *x = static_cast<const uint16_t *>(in.p[wl]);
        for (int c = threadIdx.x; c < n4 / 2; c += kThreads) {
            const uint64_t j = j0 + (uint64_t)c * 8;
            if (j >= d) break;
            uint32_t w[4] = {0u, 0u, 0u, 0u};
            if (j + 8 <= d) {
                const uint4 q = __ldg(reinterpret_cast<const uint4 *>(x + j));
                w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w;
            } else {
                for (int e = 0; e < 8; ++e)
                    if (j + e < d) w[e >> 1] |= (uint32_t)__ldg(x + j + e) << ((e & 1) * 16);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const double lo = (double)__uint_as_float(w[q] << 16);
                const double hi = (double)__uint_as_float(w[q] & 0xFFFF0000u);
                s = fma(lo, lo, s);
                s = fma(hi, hi, s);
            }
        }
    } else {
        for (int c = threadIdx.x; c < n4; c += kThreads) {
            const uint64_t j = j0 + (uint64_t)c * 4;
            if (j >= d) break;
            const float4 v = load_f32x4_masked(static_cast<const float *>(in.p[wl]), j, d);
            s = fma((double)v.x, (double)v.x, s);
            s = fma((double)v.y, (double)v.y, s);
            s = fma((double)v.z, (double)v.z, s);
            s = fma((double)v.w, (double)v.w, s);
        }
    }
    __shared__ double red[kThreads / 32];
    for (int off = 16; off > 0; off >>= 1) s += __shfl_down_sync(0xFFFFFFFFu, s, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < kThreads / 32; ++w) t += red[w];
        partial[(uint64_t)wl * chunks_per_worker + chunk] = t;
    }
}

// M per block from the partial sums (Section 5.3: M = t_p * max_i ||x_i|| / sqrt(B)).  One warp
// per RHT block, eight workers at a time with four lanes per worker: a lane adds every fourth
// partial sum of its worker (loads independent of each other), the four lanes are combined,
// one square root per worker, then the maximum over workers.  The order is fixed, so the
// result does not depend on timing.
__global__ void __launch_bounds__(128)
prepare_final_kernel(const double *__restrict__ partial, uint32_t n, uint64_t nblocks,
                     uint64_t chunks_per_block, uint64_t chunks_per_worker, double t_p, uint32_t k,
                     float *__restrict__ scales, DeviceBlock *dev)
{
    const uint64_t blk = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (blk >= nblocks) return;
    double ell = 0.0;
    for (uint32_t i0 = 0; i0 < n; i0 += 8u) {
        const uint32_t i = i0 + ((uint32_t)lane >> 2);
        const bool live = i < n;
        const double *p = partial + (uint64_t)(live ? i : 0u) * chunks_per_worker + blk * chunks_per_block;
        double s = 0.0;
        for (uint64_t c = (uint64_t)(lane & 3); c < chunks_per_block; c += 4) s += p[c];
        s += __shfl_xor_sync(0xFFFFFFFFu, s, 1);
        s += __shfl_xor_sync(0xFFFFFFFFu, s, 2);
        double norm = live ? sqrt(s) : 0.0;
        for (int off = 4; off < 32; off <<= 1) {
            const double other = __shfl_xor_sync(0xFFFFFFFFu, norm, off);
            if (other > norm || other != other) norm = other;      // a NaN norm sticks
        }
        if (norm > ell || norm != norm) ell = norm;
    }
    if (lane != 0) return;
    float M = (float)(t_p * ell / sqrt((double)((uint64_t)1 << k)));
    uint32_t flags = 0;
    if (!isfinite(M)) { M = 0.0f; flags |= THC_STATUS_NONFINITE; }
    if (M == 0.0f) flags |= THC_STATUS_ZERO_BLOCK;
    scales[blk] = M;
    if (flags) atomicOr(&dev->status, flags);
}

// Exact range (Algorithm 1's preliminary stage on the rotated coordinates): keys start at
// (+max, 0); afterwards they become nblocks minima followed by nblocks maxima in `scales`.
// A block with a non-finite rotated coordinate gets (0, 0) and THC_STATUS_NONFINITE.
__global__ void range_init_kernel(uint32_t *keys, uint64_t nblocks)
{
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < nblocks) { keys[i] = 0xFFFFFFFFu; keys[nblocks + i] = 0u; }
}

__global__ void range_final_kernel(const uint32_t *keys, uint64_t nblocks, float *scales, DeviceBlock *dev)
{
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nblocks) return;
    float lo = key_float(keys[i]), hi = key_float(keys[nblocks + i]);
    uint32_t flags = 0;
    if (!isfinite(lo) || !isfinite(hi)) { lo = 0.0f; hi = 0.0f; flags |= THC_STATUS_NONFINITE; }
    if (hi == 0.0f && lo == 0.0f) flags |= THC_STATUS_ZERO_BLOCK;   // a constant block decodes exactly
    scales[i] = lo;
    scales[nblocks + i] = hi;
    if (flags) atomicOr(&dev->status, flags);
}

// ---------------------------------------------------------------------------- aggregate
// Y[j] = sum_i T[z_i[j]] (Algorithm 2, PS line).  One thread per 32 coordinates.
template <int BITS, int W>
__global__ void __launch_bounds__(kThreads)
aggregate_kernel(PtrArray in, uint32_t n, uint64_t units, uint64_t d_pad, const DeviceBlock *dev,
                 unsigned char *__restrict__ sum)
{
    __shared__ uint32_t T[256];
    for (int z = threadIdx.x; z < (1 << BITS); z += kThreads) T[z] = dev->table[z];
    __syncthreads();
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        // coordinates past the last whole group of 32 (blocks of 8 or 16 coordinates only)
        for (uint64_t j = units * 32; j < d_pad; ++j) {
            uint32_t acc = 0;
            for (uint32_t i = 0; i < n; ++i) {
                const unsigned char *pb = static_cast<const unsigned char *>(in.p[i]);
                const uint64_t bit = j * BITS;
                uint32_t two = pb[bit >> 3];
                if (((bit & 7) + BITS) > 8) two |= (uint32_t)pb[(bit >> 3) + 1] << 8;
                acc += T[(two >> (bit & 7)) & ((1u << BITS) - 1u)];
            }
            if constexpr (W == 8) sum[j] = (unsigned char)acc;
            else if constexpr (W == 16) reinterpret_cast<uint16_t *>(sum)[j] = (uint16_t)acc;
            else reinterpret_cast<uint32_t *>(sum)[j] = acc;
        }
    }
    constexpr int kInWords = BITS;                 // 32 indices * BITS bits = BITS words
    for (uint64_t u = (uint64_t)blockIdx.x * kThreads + threadIdx.x; u < units;
         u += (uint64_t)gridDim.x * kThreads) {
        uint32_t acc[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) acc[e] = 0;
        for (uint32_t i = 0; i < n; ++i) {
            const uint32_t *src = reinterpret_cast<const uint32_t *>(
                static_cast<const unsigned char *>(in.p[i]) + u * (4 * BITS));
            uint32_t w[kInWords];
            if constexpr (BITS == 8) {
                const uint4 a = __ldg(reinterpret_cast<const uint4 *>(src));
                const uint4 b = __ldg(reinterpret_cast<const uint4 *>(src) + 1);
                w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
                w[4] = b.x; w[5] = b.y; w[6] = b.z; w[7] = b.w;
            } else if constexpr (BITS == 4) {
                const uint4 a = __ldg(reinterpret_cast<const uint4 *>(src));
                w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
            } else if constexpr (BITS == 3) {
                w[0] = __ldg(src); w[1] = __ldg(src + 1); w[2] = __ldg(src + 2);
            } else if constexpr (BITS == 2) {
                const uint2 a = __ldg(reinterpret_cast<const uint2 *>(src));
                w[0] = a.x; w[1] = a.y;
            } else {
                w[0] = __ldg(src);
            }
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                const int bit = e * BITS;
                // a 3-bit index may straddle two words: funnel shift over the pair
                const uint32_t lo = w[bit >> 5], hi = w[((bit >> 5) + 1) < kInWords ? (bit >> 5) + 1 : (bit >> 5)];
                const uint32_t z = __funnelshift_r(lo, hi, bit & 31) & ((1u << BITS) - 1u);
                acc[e] += T[z];
            }
        }
        unsigned char *dst = sum + u * (32 * W / 8);
        if constexpr (W == 8) {
            uint32_t o[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
                o[q] = (acc[4 * q] & 0xFFu) | ((acc[4 * q + 1] & 0xFFu) << 8) |
                       ((acc[4 * q + 2] & 0xFFu) << 16) | (acc[4 * q + 3] << 24);
            reinterpret_cast<uint4 *>(dst)[0] = make_uint4(o[0], o[1], o[2], o[3]);
            reinterpret_cast<uint4 *>(dst)[1] = make_uint4(o[4], o[5], o[6], o[7]);
        } else if constexpr (W == 16) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t o[4];
#pragma unroll
                for (int t = 0; t < 4; ++t)
                    o[t] = (acc[8 * q + 2 * t] & 0xFFFFu) | (acc[8 * q + 2 * t + 1] << 16);
                reinterpret_cast<uint4 *>(dst)[q] = make_uint4(o[0], o[1], o[2], o[3]);
            }
        } else {
#pragma unroll
            for (int q = 0; q < 8; ++q)
                reinterpret_cast<uint4 *>(dst)[q] =
                    make_uint4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]);
        }
    }
}

}  // namespace thc

#include "thc_pipeline.cuh"

// =========================================================================== host side
using namespace thc;

struct thc_ctx {
    thc_config cfg;
    uint32_t acc_bits;
    bool identity;
    int device;                 // -1: no CUDA device, host-only context
    DeviceBlock *dev;
    PhiloxKeys keys;
    uint32_t lut_rep;
    int sm_count;
    // Encoded tensor maps of recent launches, keyed by what they describe: a training loop calls
    // with the same buffers every step, and encoding up to n + 1 maps per call costs more host
    // time than a small launch takes on the device.
    struct MapEntry { const void *base; uint64_t cols, rows, pitch; uint32_t box_rows, box_cols, half, groups; CUtensorMap map; };
    static constexpr int kMapCache = 2 * (THC_MAX_WORKERS + 2);
    mutable MapEntry map_cache[kMapCache];
    mutable int map_cache_used, map_cache_next;
    mutable std::mutex map_mutex;
};

static thread_local cudaError_t g_last_cuda = cudaSuccess;
static thread_local char g_err_text[256];

static int cuda_fail(cudaError_t e)
{
    g_last_cuda = e;
    return THC_ECUDA;
}

#define THC_CUDA(call)                                        \
    do {                                                      \
        cudaError_t e__ = (call);                             \
        if (e__ != cudaSuccess) return cuda_fail(e__);        \
    } while (0)

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

const char *thc_version(void) { return "thc-b200 0.1 (sm_100a)"; }

const char *thc_strerror(int code)
{
    switch (code) {
    case THC_OK: return "ok";
    case THC_EINVAL: return "invalid configuration or argument";
    case THC_EUNSUPPORTED: return "unsupported configuration";
    case THC_EWORKSPACE: return "workspace too small (see thc_sizes)";
    case THC_ECUDA:
        if (g_last_cuda == cudaSuccess) return "CUDA error: context has no device";
        snprintf(g_err_text, sizeof g_err_text, "CUDA error: %s", cudaGetErrorString(g_last_cuda));
        return g_err_text;
    default: return "unknown error code";
    }
}

static int validate_config(const thc_config *c, uint32_t *acc_bits, bool *identity)
{
    if (c == nullptr) return THC_EINVAL;
    if (!(c->bits == 1 || c->bits == 2 || c->bits == 3 || c->bits == 4 || c->bits == 8)) return THC_EINVAL;
    const uint32_t levels = 1u << c->bits;
    if (c->granularity < levels - 1) return THC_EINVAL;
    if (c->granularity > 255) return THC_EUNSUPPORTED;
    if (c->table[0] != 0 || c->table[levels - 1] != c->granularity) return THC_EINVAL;
    for (uint32_t z = 0; z + 1 < levels; ++z)
        if (c->table[z + 1] <= c->table[z]) return THC_EINVAL;
    if (!(c->t_p > 0.0) || !isfinite(c->t_p)) return THC_EINVAL;
    if (c->log2_block < 3 || c->log2_block > 22) return THC_EINVAL;
    if (c->in_dtype != THC_F32 && c->in_dtype != THC_BF16) return THC_EINVAL;
    if (c->workers == 0 || c->workers > THC_MAX_WORKERS) return THC_EINVAL;
    if (c->range_mode != THC_RANGE_NORM && c->range_mode != THC_RANGE_MINMAX) return THC_EINVAL;
    if (c->range_mode == THC_RANGE_MINMAX && c->in_dtype != THC_F32) return THC_EUNSUPPORTED;
    const uint64_t max_sum = (uint64_t)c->workers * c->granularity;
    uint32_t w = c->acc_bits;
    if (w == 0) w = max_sum <= 0xFFu ? 8 : max_sum <= 0xFFFFu ? 16 : 32;
    if (!(w == 8 || w == 16 || w == 32)) return THC_EINVAL;
    if (w < 32 && max_sum > ((1ull << w) - 1)) return THC_EINVAL;
    *acc_bits = w;
    bool id = c->granularity == levels - 1;
    for (uint32_t z = 0; id && z < levels; ++z) id = c->table[z] == z;
    *identity = id;
    return THC_OK;
}

int thc_create(const thc_config *cfg, thc_ctx **out)
{
    if (out == nullptr) return THC_EINVAL;
    *out = nullptr;
    uint32_t acc_bits = 0;
    bool identity = false;
    const int rc = validate_config(cfg, &acc_bits, &identity);
    if (rc != THC_OK) return rc;
    thc_ctx *ctx = new (std::nothrow) thc_ctx;
    if (ctx == nullptr) return THC_EINVAL;
    ctx->cfg = *cfg;
    ctx->acc_bits = acc_bits;
    ctx->identity = identity;
    ctx->device = -1;
    ctx->dev = nullptr;
    ctx->sm_count = 148;
    ctx->map_cache_used = 0;
    ctx->map_cache_next = 0;
    uint32_t k0 = (uint32_t)cfg->seed, k1 = (uint32_t)(cfg->seed >> 32);
    for (int r = 0; r < 10; ++r) {
        ctx->keys.k[2 * r] = k0;
        ctx->keys.k[2 * r + 1] = k1;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    const uint32_t g = cfg->granularity;
    ctx->lut_rep = 8;

    // host copy of the device block
    DeviceBlock *h = new (std::nothrow) DeviceBlock;
    if (h == nullptr) { delete ctx; return THC_EINVAL; }
    memset(h, 0, sizeof *h);
    const uint32_t levels = 1u << cfg->bits;
    for (uint32_t z = 0; z < levels; ++z) h->table[z] = cfg->table[z];
    for (uint32_t f = 0; f <= g; ++f) {
        const uint32_t ff = f < g ? f : g - 1;            // u = 1 falls in the last interval
        uint32_t z0 = 0;
        while (z0 + 1 <= levels - 2 && cfg->table[z0 + 1] <= ff) ++z0;
        const float ntf = -(float)cfg->table[z0];
        const float r16 = 65536.0f / (float)(cfg->table[z0 + 1] - cfg->table[z0]);
        uint32_t b0, b1;
        memcpy(&b0, &ntf, 4);
        memcpy(&b1, &r16, 4);
        h->lut[f] = make_uint4(b0, b1, z0, 0u);
    }

    int count = 0;
    if (cudaGetDeviceCount(&count) == cudaSuccess && count > 0) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void **>(&ctx->dev), sizeof(DeviceBlock));
        if (e == cudaSuccess) e = cudaMemcpy(ctx->dev, h, sizeof(DeviceBlock), cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) {
            if (ctx->dev) cudaFree(ctx->dev);
            delete h;
            delete ctx;
            return cuda_fail(e);
        }
        ctx->device = dev;
    } else {
        (void)cudaGetLastError();   // no device: host-only context
    }
    delete h;
    *out = ctx;
    return THC_OK;
}

int thc_destroy(thc_ctx *ctx)
{
    if (ctx == nullptr) return THC_OK;
    if (ctx->dev != nullptr) cudaFree(ctx->dev);
    delete ctx;
    return THC_OK;
}

static uint64_t round_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

// Schedule of the persistent pipeline for `wb_count` worker-blocks of 2^k coordinates:
// how far pass B trails pass A (lag, in worker-blocks) and how many ring slots that needs.
struct PipePlan { uint32_t grid, lag, ring; };

static PipePlan plan_pipeline(const thc_ctx *ctx, uint64_t wb_count)
{
    const uint32_t k = ctx->cfg.log2_block;
    const uint64_t T = 1ull << (k - kPLog2);
    const uint64_t resident = (uint64_t)ctx->sm_count * 3;
    PipePlan p;
    const uint64_t tasks = wb_count * T * 2;
    p.grid = (uint32_t)(tasks < resident ? tasks : resident);
    // tasks in flight: per CTA one running, one handed over, and at times one being claimed
    const uint64_t inflight = resident * 5 / 2;
    uint64_t lag = (inflight + 2 * T - 1) / (2 * T) + 1;
    uint64_t ring = lag + (inflight + 2 * T - 1) / (2 * T) + 1;
    if (lag > wb_count) lag = wb_count;
    if (ring > wb_count) ring = wb_count;
    if (ring > (uint64_t)kMaxRing) {           // tiny blocks on a huge grid: shrink the window
        ring = kMaxRing;
        if (lag > ring - 2) lag = ring - 2;
    }
    p.lag = (uint32_t)lag;
    p.ring = (uint32_t)ring;
    return p;
}

// The same for the fused-scales kernel: pass B of a block can start only when all n workers'
// tiles of the block are done, so it trails by n - 1 more worker-blocks and the ring grows by
// as many slots.  Used only where that ring still fits comfortably in L2 and the per-block
// counters (16 residues) cannot alias; otherwise the caller runs prepare and compress apart.
static bool plan_pipeline_fused(const thc_ctx *ctx, uint64_t nblocks, uint32_t n, PipePlan *out)
{
    if (ctx->cfg.log2_block != 20 || ctx->cfg.in_dtype != THC_F32) return false;
    if (ctx->cfg.range_mode != THC_RANGE_NORM) return false;
    const uint64_t wb_count = nblocks * n;
    PipePlan p = plan_pipeline(ctx, wb_count);
    const uint64_t window = p.ring - p.lag;
    const uint64_t lag = (uint64_t)p.lag + n - 1;
    const uint64_t ring = lag + window;
    if (ring > wb_count || ring > (uint64_t)kMaxRing) return false;
    if (ring * ((uint64_t)4 << 20) > ((uint64_t)96 << 20)) return false;
    if ((ring + n - 1) / n + 2 > 16) return false;
    p.lag = (uint32_t)lag;
    p.ring = (uint32_t)ring;
    *out = p;
    return true;
}

// Workspace a pipeline launch over `wb_count` worker-blocks really touches when it computes no
// scales: the ring and, behind it, one word pair per block for the exact-range keys.
static uint64_t pipeline_workspace_need(const thc_ctx *ctx, uint64_t nblocks, uint64_t wb_count)
{
    const PipePlan pl = plan_pipeline(ctx, wb_count);
    return ((uint64_t)pl.ring << ctx->cfg.log2_block) * 4 + nblocks * 8;
}

int thc_sizes(const thc_ctx *ctx, uint64_t d, uint32_t n_local, thc_sizes_t *s)
{
    if (ctx == nullptr || s == nullptr || d == 0 || n_local == 0 || n_local > THC_MAX_WORKERS)
        return THC_EINVAL;
    const uint32_t k = ctx->cfg.log2_block;
    const uint64_t B = 1ull << k;
    if (d > (1ull << 40)) return THC_EINVAL;
    memset(s, 0, sizeof *s);
    s->d_pad = round_up(d, B);
    s->nblocks = s->d_pad / B;
    s->packed_bytes = s->d_pad * ctx->cfg.bits / 8;
    s->sum_bytes = s->d_pad * ctx->acc_bits / 8;
    s->rotated_bytes = s->d_pad * 4;
    s->acc_bits = ctx->acc_bits;
    s->scales_count = ctx->cfg.range_mode == THC_RANGE_MINMAX ? 2 * s->nblocks : s->nblocks;
    const uint32_t chunk_log2 = k < (uint32_t)kTileLog2 ? k : (uint32_t)kTileLog2;
    const uint64_t prepare_ws = (uint64_t)n_local * (s->d_pad >> chunk_log2) * 8;
    uint64_t two_pass_ws = 0;
    if (k > (uint32_t)kTileLog2) {
        const PipePlan pl = plan_pipeline(ctx, s->nblocks * n_local);
        two_pass_ws = (uint64_t)pl.ring * B * 4 + s->nblocks * 8;       // + range keys
        PipePlan pf;
        if (plan_pipeline_fused(ctx, s->nblocks, n_local, &pf)) {
            const uint64_t fused_ws = (uint64_t)pf.ring * B * 4 + s->nblocks * n_local * (B >> kPLog2) * 8 +
                                      s->nblocks * 8;       // ring, tile sums, per-block quantiser constants
            if (fused_ws > two_pass_ws) two_pass_ws = fused_ws;
            s->fused_scales = 1;
        }
    }
    // scratch of prepare / the pipeline's ring, then one worker's table values (error feedback)
    s->workspace_bytes = round_up((prepare_ws > two_pass_ws ? prepare_ws : two_pass_ws) + 256, 256) +
                         round_up(s->sum_bytes, 256);
    return THC_OK;
}

static int check_launch_ctx(const thc_ctx *ctx)
{
    if (ctx == nullptr) return THC_EINVAL;
    if (ctx->device < 0 || ctx->dev == nullptr) { g_last_cuda = cudaSuccess; return THC_ECUDA; }
    // the context's device block, tables and counters live on the device it was created on
    int cur = -1;
    THC_CUDA(cudaGetDevice(&cur));
    if (cur != ctx->device) return THC_EINVAL;
    return THC_OK;
}

static int check_ptr_array(const void *const *arr, uint32_t n)
{
    if (arr == nullptr) return THC_EINVAL;
    for (uint32_t i = 0; i < n; ++i)
        if (arr[i] == nullptr || !aligned16(arr[i])) return THC_EINVAL;
    return THC_OK;
}

int thc_prepare(thc_ctx *ctx, const void *const *grads, uint32_t n, uint64_t d, float *scales,
                void *workspace, uint64_t workspace_bytes, void *stream)
{
    int rc = check_launch_ctx(ctx);
    if (rc != THC_OK) return rc;
    thc_sizes_t sz;
    if ((rc = thc_sizes(ctx, d, n, &sz)) != THC_OK) return rc;
    if ((rc = check_ptr_array(grads, n)) != THC_OK) return rc;
    if (scales == nullptr || workspace == nullptr || !aligned16(workspace)) return THC_EINVAL;
    if (workspace_bytes < sz.workspace_bytes) return THC_EWORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint32_t k = ctx->cfg.log2_block;
    if (ctx->cfg.range_mode == THC_RANGE_MINMAX) return THC_EUNSUPPORTED;   // thc_prepare_minmax
    const uint32_t chunk_log2 = k < (uint32_t)kTileLog2 ? k : (uint32_t)kTileLog2;
    const uint64_t chunks_per_worker = sz.d_pad >> chunk_log2;
    const uint64_t chunks_per_block = 1ull << (k - chunk_log2);
    if (chunks_per_worker > 0x7FFFFFFFull) return THC_EUNSUPPORTED;
    PtrArray in;
    memset(&in, 0, sizeof in);
    for (uint32_t i = 0; i < n; ++i) in.p[i] = grads[i];
    double *partial = static_cast<double *>(workspace);
    const dim3 grid((unsigned)chunks_per_worker, n);
    if (ctx->cfg.in_dtype == THC_BF16)
        prepare_partial_kernel<true><<<grid, kThreads, 0, st>>>(in, d, chunk_log2, chunks_per_worker, partial);
    else
        prepare_partial_kernel<false><<<grid, kThreads, 0, st>>>(in, d, chunk_log2, chunks_per_worker, partial);
    THC_CUDA(cudaGetLastError());
    prepare_final_kernel<<<(unsigned)((sz.nblocks + 3) / 4), 128, 0, st>>>(
        partial, n, sz.nblocks, chunks_per_block, chunks_per_worker, ctx->cfg.t_p, k, scales, ctx->dev);
    THC_CUDA(cudaGetLastError());
    return THC_OK;
}

// ---- tile-kernel dispatch
typedef void (*tile_kernel_t)(TileGeom, PtrArray, MutPtrArray, MutPtrArray, const float *,
                              DeviceBlock *, PhiloxKeys);

template <int LOAD, int STORE>
static tile_kernel_t pick_tile_kernel(uint32_t bits, bool identity)
{
    if constexpr (STORE != kStoreQuant) {
        return rht_tile_kernel<LOAD, STORE, 4, true>;
    } else {
    switch (bits) {
    case 1: return identity ? rht_tile_kernel<LOAD, STORE, 1, true> : rht_tile_kernel<LOAD, STORE, 1, false>;
    case 2: return identity ? rht_tile_kernel<LOAD, STORE, 2, true> : rht_tile_kernel<LOAD, STORE, 2, false>;
    case 3: return identity ? rht_tile_kernel<LOAD, STORE, 3, true> : rht_tile_kernel<LOAD, STORE, 3, false>;
    case 4: return identity ? rht_tile_kernel<LOAD, STORE, 4, true> : rht_tile_kernel<LOAD, STORE, 4, false>;
    default: return identity ? rht_tile_kernel<LOAD, STORE, 8, true> : rht_tile_kernel<LOAD, STORE, 8, false>;
    }
    }
}

static size_t tile_smem_bytes(const thc_ctx *ctx, const TileGeom &g)
{
    return (size_t)kTileElems * 4 + kSignWordsMax * 4 +
           (((size_t)g.blocks_in_tile * 8 + 15) & ~(size_t)15) +
           (size_t)(ctx->cfg.granularity + 1) * kLutEntryBytes;
}

// cudaFuncSetAttribute is needed once per kernel and dynamic shared-memory size; remember
// what has been set per (kernel, device); a larger request raises the recorded size.
static int ensure_dynamic_smem(const void *kern, size_t smem)
{
    static std::mutex guard;
    std::lock_guard<std::mutex> lock(guard);
    static const void *seen_kern[96];
    static size_t seen_size[96];
    static int seen_dev[96];
    static int seen = 0;
    int dev = 0;
    THC_CUDA(cudaGetDevice(&dev));
    for (int i = 0; i < seen; ++i)
        if (seen_kern[i] == kern && seen_dev[i] == dev) {
            if (seen_size[i] >= smem) return THC_OK;
            THC_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            seen_size[i] = smem;
            return THC_OK;
        }
    THC_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    if (seen < 96) { seen_kern[seen] = kern; seen_size[seen] = smem; seen_dev[seen] = dev; ++seen; }
    return THC_OK;
}

static int launch_tile(const thc_ctx *ctx, tile_kernel_t kern, const TileGeom &g, uint64_t tiles,
                       uint32_t n_local, const PtrArray &in, const MutPtrArray &out,
                       const MutPtrArray &rot, const float *scales, cudaStream_t st)
{
    if (tiles > 0x7FFFFFFFull) return THC_EUNSUPPORTED;
    const size_t smem = tile_smem_bytes(ctx, g);
    { const int rc = ensure_dynamic_smem(reinterpret_cast<const void *>(kern), smem); if (rc != THC_OK) return rc; }
    kern<<<dim3((unsigned)tiles, n_local), kThreads, smem, st>>>(g, in, out, rot, scales, ctx->dev,
                                                                 ctx->keys);
    THC_CUDA(cudaGetLastError());
    return THC_OK;
}

static TileGeom base_geom(const thc_ctx *ctx, const thc_sizes_t &sz, uint64_t d, uint32_t round)
{
    TileGeom g;
    memset(&g, 0, sizeof g);
    g.d = d;
    g.d_pad = sz.d_pad;
    g.k = ctx->cfg.log2_block;
    g.lut_rep = ctx->lut_rep;
    g.granularity = ctx->cfg.granularity;
    g.round = round;
    g.c_block = (float)(1.0 / sqrt((double)(1ull << g.k)));
    g.exact_range = ctx->cfg.range_mode == THC_RANGE_MINMAX ? 1u : 0u;
    return g;
}

static void geom_pass_a(TileGeom &g)
{
    g.row_log2 = 0;
    g.col_log2 = kTileLog2;
    g.row_stride = 0;
    g.lo_cbit = 0;
    g.hi_cbit = (g.k < (uint32_t)kTileLog2 ? g.k : (uint32_t)kTileLog2) - 2;
    g.blocks_in_tile = g.k >= (uint32_t)kTileLog2 ? 1u : 1u << (kTileLog2 - g.k);
}

// ---- persistent pipeline dispatch (RHT blocks of 2^15 .. 2^24 coordinates)
typedef void (*pipe_kernel_t)(const TmaMaps, PipeParams, PtrArrayP, MutPtrArrayP, MutPtrArrayP, PhiloxKeys);

template <int MODE, int KB>
static pipe_kernel_t pick_pipe_kernel_kb(uint32_t bits, bool identity)
{
    if constexpr (MODE == kRangeF32) {
        return thc_pipeline_kernel<MODE, 4, true, KB>;
    } else if constexpr (MODE == kAggDecompress) {
        return thc_pipeline_kernel<MODE, 4, true, KB>;     // one launch only for 4-bit indices (see the entry point)
    } else if constexpr (MODE == kErrorFeedback) {
        switch (bits) {
        case 1: return thc_pipeline_kernel<MODE, 1, true, KB>;
        case 2: return thc_pipeline_kernel<MODE, 2, true, KB>;
        case 3: return thc_pipeline_kernel<MODE, 3, true, KB>;
        case 4: return thc_pipeline_kernel<MODE, 4, true, KB>;
        default: return thc_pipeline_kernel<MODE, 8, true, KB>;
        }
    } else if constexpr (MODE != kCompressF32 && MODE != kCompressBF16 && MODE != kCompressF32Fused) {
        return thc_pipeline_kernel<MODE, 4, true, KB>;
    } else {
        switch (bits) {
        case 1: return identity ? thc_pipeline_kernel<MODE, 1, true, KB> : thc_pipeline_kernel<MODE, 1, false, KB>;
        case 2: return identity ? thc_pipeline_kernel<MODE, 2, true, KB> : thc_pipeline_kernel<MODE, 2, false, KB>;
        case 3: return identity ? thc_pipeline_kernel<MODE, 3, true, KB> : thc_pipeline_kernel<MODE, 3, false, KB>;
        case 4: return identity ? thc_pipeline_kernel<MODE, 4, true, KB> : thc_pipeline_kernel<MODE, 4, false, KB>;
        default: return identity ? thc_pipeline_kernel<MODE, 8, true, KB> : thc_pipeline_kernel<MODE, 8, false, KB>;
        }
    }
}

// The 2^20-coordinate block (the paper's 4 MB partition) gets the compile-time geometry.
template <int MODE>
static pipe_kernel_t pick_pipe_kernel(uint32_t bits, bool identity, uint32_t k)
{
    if constexpr (MODE == kCompressF32 || MODE == kCompressBF16) {
        // 2^21 and 2^22 (the largest configuration): the generic path with its geometry fixed at
        // compile time
        // (4-bit indices only, the width of every benchmark configuration with such blocks: each
        // further instantiation costs build time)
        if (k == 21 && bits == 4)
            return identity ? thc_pipeline_kernel<MODE, 4, true, 8> : thc_pipeline_kernel<MODE, 4, false, 8>;
        if (k == 22 && bits == 4)
            return identity ? thc_pipeline_kernel<MODE, 4, true, 9> : thc_pipeline_kernel<MODE, 4, false, 9>;
    }
    return k == 20 ? pick_pipe_kernel_kb<MODE, 7>(bits, identity)
                   : pick_pipe_kernel_kb<MODE, 0>(bits, identity);
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda).
typedef CUresult (*encode_tiled_t)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                   const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static encode_tiled_t get_encode_tiled()
{
    static const encode_tiled_t fn = []() -> encode_tiled_t {     // initialised once, thread-safe
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            return reinterpret_cast<encode_tiled_t>(p);
        return nullptr;
    }();
    return fn;
}

// A 2-D map over `rows` rows of `cols` 32-bit words (row pitch in bytes), box box_cols x
// box_rows (32 columns with the 128-byte swizzle, 16 with the 64-byte one).  The data type is
// UINT32 so that bits travel unchanged.
// With box_groups > 0 the rows are seen as cols / 32 groups of 32 words and the map is 3-D
// (word in group, group, row) with a box of 32 x box_groups x box_rows: one copy then brings
// box_rows rows of 32 * box_groups words each, and they land densely, row after row, in the
// 128-byte swizzle (16-byte chunk c at c ^ ((c >> 3) & 7)).
static int encode_map(CUtensorMap *map, const void *base, uint64_t cols, uint64_t rows,
                      uint64_t pitch_bytes, uint32_t box_rows, uint32_t box_cols = 32u, bool half_words = false,
                      uint32_t box_groups = 0u)
{
    encode_tiled_t enc = get_encode_tiled();
    if (enc == nullptr) return THC_ECUDA;
    if (box_groups != 0u) {
        const cuuint64_t dims3[3] = {32u, cols / 32u, rows};
        const cuuint64_t strides3[2] = {128u, pitch_bytes};
        const cuuint32_t box3[3] = {32u, box_groups, box_rows};
        const cuuint32_t estr3[3] = {1u, 1u, 1u};
        const CUresult r3 = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<void *>(base), dims3, strides3,
                                box3, estr3, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        return r3 == CUDA_SUCCESS ? THC_OK : THC_ECUDA;
    }
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {pitch_bytes};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    // 16-bit elements (bf16 gradients as rows of 32: 64 bytes) or 32-bit words; rows of 64
    // bytes take the 64-byte swizzle
    const bool rows64 = half_words ? box_cols == 32u : box_cols == 16u;
    const CUresult r = enc(map, half_words ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : CU_TENSOR_MAP_DATA_TYPE_UINT32, 2,
                           const_cast<void *>(base), dims, strides,
                           box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           rows64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? THC_OK : THC_ECUDA;
}

// encode_map through the context's cache.
static int cached_map(const thc_ctx *ctx, CUtensorMap *map, const void *base, uint64_t cols, uint64_t rows,
                      uint64_t pitch_bytes, uint32_t box_rows, uint32_t box_cols = 32u, bool half_words = false,
                      uint32_t box_groups = 0u)
{
    std::lock_guard<std::mutex> lock(ctx->map_mutex);
    for (int i = 0; i < ctx->map_cache_used; ++i) {
        const thc_ctx::MapEntry &e = ctx->map_cache[i];
        if (e.base == base && e.cols == cols && e.rows == rows && e.pitch == pitch_bytes && e.box_rows == box_rows &&
            e.box_cols == box_cols && e.half == (half_words ? 1u : 0u) && e.groups == box_groups) {
            *map = e.map;
            return THC_OK;
        }
    }
    const int rc = encode_map(map, base, cols, rows, pitch_bytes, box_rows, box_cols, half_words, box_groups);
    if (rc != THC_OK) return rc;
    int slot = ctx->map_cache_used < thc_ctx::kMapCache ? ctx->map_cache_used++ : ctx->map_cache_next;
    ctx->map_cache_next = (slot + 1) % thc_ctx::kMapCache;
    thc_ctx::MapEntry &e = ctx->map_cache[slot];
    e.base = base; e.cols = cols; e.rows = rows; e.pitch = pitch_bytes; e.box_rows = box_rows; e.box_cols = box_cols;
    e.half = half_words ? 1u : 0u; e.groups = box_groups; e.map = *map;
    return THC_OK;
}

static int launch_pipeline(const thc_ctx *ctx, pipe_kernel_t kern, bool compress_f32,
                           const thc_sizes_t &sz, uint64_t d, uint32_t n_local, uint32_t worker_base, uint32_t round, uint32_t divisor,
                           const float *scales, void *workspace, const PtrArrayP &in,
                           const MutPtrArrayP &out, const MutPtrArrayP &rot, cudaStream_t st,
                           float *fused_scales_out = nullptr, bool compress_bf16 = false, uint32_t agg_n = 0)
{
    const uint32_t k = ctx->cfg.log2_block;
    PipeParams P;
    memset(&P, 0, sizeof P);
    P.d = d;
    P.d_pad = sz.d_pad;
    P.wb_count = sz.nblocks * n_local;
    const uint64_t T = 1ull << (k - kPLog2);
    P.total_tasks = P.wb_count * T * 2;
    if (P.wb_count >= 0x7FFFFFFFull || P.total_tasks >= 0x7FFFFFFFull) return THC_EUNSUPPORTED;
    PipePlan pl = plan_pipeline(ctx, P.wb_count);
    // Compress of 2^22 blocks: pass B trails by two worker-blocks in a ring of four slots
    // (64 MB stay in L2 better than the planned six slots of 16 MB; the workspace holds those).
    // The exact-range keys stay where the planned ring ends: thc_prepare_minmax looks there.
    const uint32_t planned_ring = pl.ring;
    if ((compress_f32 || compress_bf16) && k == 22 && pl.ring > 4) { pl.lag = 2; pl.ring = 4; }
    if (fused_scales_out != nullptr) {
        if (!plan_pipeline_fused(ctx, sz.nblocks, n_local, &pl)) return THC_EUNSUPPORTED;
        P.tile_sq = reinterpret_cast<double *>(static_cast<unsigned char *>(workspace) +
                                               ((uint64_t)pl.ring << k) * 4);
        P.fused_const = reinterpret_cast<float2 *>(P.tile_sq + P.wb_count * T);
        P.scales_out = fused_scales_out;
        P.t_p = ctx->cfg.t_p;
    }
    P.ring = static_cast<float *>(workspace);
    P.scales = scales;
    P.dev = ctx->dev;
    P.k = k;
    P.kb = k - kPLog2;
    P.n_local = n_local;
    P.lag = pl.lag;
    P.ring_slots = pl.ring;
    P.granularity = ctx->cfg.granularity;
    P.divisor = divisor;
    P.round = round;
    P.worker_base = worker_base;
    P.c_block = (float)(1.0 / sqrt((double)(1ull << k)));
    P.exact_range = ctx->cfg.range_mode == THC_RANGE_MINMAX ? 1u : 0u;
    P.nblocks = (uint32_t)sz.nblocks;
    P.agg_n = agg_n;
    P.agg_acc_bits = ctx->acc_bits;
    P.range_keys = reinterpret_cast<uint32_t *>(static_cast<unsigned char *>(workspace) +
                                                ((uint64_t)planned_ring << k) * 4);
    const uint64_t nblk_cached = sz.nblocks < (uint64_t)kBlockConstMax ? sz.nblocks : (uint64_t)kBlockConstMax;
    const size_t smem = (size_t)1024 + (size_t)2 * kPElems * 4 + kPSignWords * 4 +
                        (size_t)(ctx->cfg.granularity + 1) * kLutEntryBytes + (size_t)nblk_cached * 8;
    { const int rc = ensure_dynamic_smem(reinterpret_cast<const void *>(kern), smem); if (rc != THC_OK) return rc; }
    // Tensor maps: the ring (pass-B panels are fetched by TMA at every block size) and, for fp32 compress, every
    // worker's gradient viewed as rows of 32 floats (whole rows only; a ragged last tile is
    // loaded by the compute warps).
    TmaMaps maps;
    memset(&maps, 0, sizeof maps);
    P.b_swz_mask = 7u;
    if (k == 20) {
        const int rc = cached_map(ctx, &maps.ring, workspace, (uint64_t)kPElems,
                                  (uint64_t)pl.ring << (k - kPLog2), (uint64_t)kPElems * 4, 128u);
        if (rc != THC_OK) return rc;
    } else if (k == 22) {
        // panels of 512 rows x 16 columns: boxes of 16 x 256, 64-byte swizzle
        const int rc = cached_map(ctx, &maps.ring, workspace, (uint64_t)kPElems,
                                  (uint64_t)pl.ring << (k - kPLog2), (uint64_t)kPElems * 4, 256u, 16u);
        if (rc != THC_OK) return rc;
        P.b_swz_mask = 3u;
        P.b_tma = 2u;
    } else if (k == 21) {
        const int rc = cached_map(ctx, &maps.ring, workspace, (uint64_t)kPElems,
                                  (uint64_t)pl.ring << (k - kPLog2), (uint64_t)kPElems * 4, 256u);
        if (rc != THC_OK) return rc;
        P.b_tma = 1u;
    } else {
        // k = 15 .. 19: panels of 2^(k-13) rows x 2^(26-k) columns, one 3-D box each
        const uint32_t kb = k - kPLog2;
        const int rc = cached_map(ctx, &maps.ring, workspace, (uint64_t)kPElems,
                                  (uint64_t)pl.ring << kb, (uint64_t)kPElems * 4, 1u << kb, 32u, false, 1u << (8u - kb));
        if (rc != THC_OK) return rc;
        P.b_tma = 3u;
    }
    if (compress_f32 && (d >> 5) >= 256) {
        for (uint32_t i = 0; i < n_local; ++i) {
            const int rc = cached_map(ctx, &maps.in[i], in.p[i], 32u, d >> 5, 128u, 256u);
            if (rc != THC_OK) return rc;
        }
    }
    if (compress_bf16 && (d >> 5) >= 256) {
        for (uint32_t i = 0; i < n_local; ++i) {
            const int rc = cached_map(ctx, &maps.in[i], in.p[i], 32u, d >> 5, 64u, 256u, 32u, true);
            if (rc != THC_OK) return rc;
        }
    }
    kern<<<pl.grid, kPCtaThreads, smem, st>>>(maps, P, in, out, rot, ctx->keys);
    THC_CUDA(cudaGetLastError());
    return THC_OK;
}

// thc_prepare in exact-range mode (Algorithm 1's preliminary stage on the rotated coordinates):
// one transform pass over all workers whose epilogue only takes the minimum and maximum, then
// the keys become the (lo, hi) planes of `scales`.  This costs about as much as the transform
// half of thc_compress: the price of a range that clamps nothing.
int thc_prepare_minmax(thc_ctx *ctx, const void *const *grads, uint32_t n, uint64_t d, uint32_t round,
                       float *scales, float *const *rotated, void *workspace, uint64_t workspace_bytes,
                       void *stream)
{
    int rc0 = check_launch_ctx(ctx);
    if (rc0 != THC_OK) return rc0;
    if (ctx->cfg.range_mode != THC_RANGE_MINMAX) return THC_EUNSUPPORTED;
    thc_sizes_t sz;
    if ((rc0 = thc_sizes(ctx, d, n, &sz)) != THC_OK) return rc0;
    if ((rc0 = check_ptr_array(grads, n)) != THC_OK) return rc0;
    if (scales == nullptr || workspace == nullptr || !aligned16(workspace)) return THC_EINVAL;
    if (workspace_bytes < sz.workspace_bytes) return THC_EWORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint32_t k = ctx->cfg.log2_block;
    const bool two_pass = k > (uint32_t)kTileLog2;
    uint32_t *keys = static_cast<uint32_t *>(workspace);
    if (two_pass) {
        const PipePlan pl = plan_pipeline(ctx, sz.nblocks * n);
        keys = reinterpret_cast<uint32_t *>(static_cast<unsigned char *>(workspace) + ((uint64_t)pl.ring << k) * 4);
    }
    const unsigned init_blocks = (unsigned)((sz.nblocks + 255) / 256);
    range_init_kernel<<<init_blocks, 256, 0, st>>>(keys, sz.nblocks);
    THC_CUDA(cudaGetLastError());
    int rc;
    if (!two_pass) {
        PtrArray in;
        MutPtrArray out, rot;
        memset(&in, 0, sizeof in);
        memset(&out, 0, sizeof out);
        memset(&rot, 0, sizeof rot);
        for (uint32_t i = 0; i < n; ++i) {
            in.p[i] = grads[i];
            if (rotated != nullptr && rotated[i] != nullptr) {
                if (!aligned16(rotated[i])) return THC_EINVAL;
                rot.p[i] = rotated[i];
            }
        }
        out.p[0] = keys;
        TileGeom g = base_geom(ctx, sz, d, round);
        geom_pass_a(g);
        const uint64_t tiles = (sz.d_pad + kTileElems - 1) / kTileElems;
        rc = launch_tile(ctx, pick_tile_kernel<kLoadGradF32, kStoreRange>(4, true), g, tiles, n, in, out, rot,
                         scales, st);
    } else {
        PtrArrayP pin;
        MutPtrArrayP pout, prot;
        memset(&pin, 0, sizeof pin);
        memset(&pout, 0, sizeof pout);
        memset(&prot, 0, sizeof prot);
        for (uint32_t i = 0; i < n; ++i) {
            pin.p[i] = grads[i];
            if (rotated != nullptr && rotated[i] != nullptr) {
                if (!aligned16(rotated[i])) return THC_EINVAL;
                prot.p[i] = rotated[i];
            }
        }
        rc = launch_pipeline(ctx, pick_pipe_kernel<kRangeF32>(4, true, k), true, sz, d, n, 0, round,
                             1, scales, workspace, pin, pout, prot, st);
    }
    if (rc != THC_OK) return rc;
    range_final_kernel<<<init_blocks, 256, 0, st>>>(keys, sz.nblocks, scales, ctx->dev);
    THC_CUDA(cudaGetLastError());
    return THC_OK;
}

int thc_compress(thc_ctx *ctx, const void *const *grads, uint32_t n_local, uint32_t worker_base,
                 uint64_t d, uint32_t round, const float *scales, void *const *packed,
                 float *const *rotated, void *workspace, uint64_t workspace_bytes, void *stream)
{
    int rc = check_launch_ctx(ctx);
    if (rc != THC_OK) return rc;
    thc_sizes_t sz;
    if ((rc = thc_sizes(ctx, d, n_local, &sz)) != THC_OK) return rc;
    if ((rc = check_ptr_array(grads, n_local)) != THC_OK) return rc;
    if ((rc = check_ptr_array(packed, n_local)) != THC_OK) return rc;
    if (scales == nullptr) return THC_EINVAL;
    if ((uint64_t)worker_base + n_local > 0xFFFFFFFFull) return THC_EINVAL;
    const uint32_t k = ctx->cfg.log2_block;
    const bool two_pass = k > (uint32_t)kTileLog2;
    if (two_pass) {
        if (workspace == nullptr || !aligned16(workspace)) return THC_EINVAL;
        if (workspace_bytes < sz.workspace_bytes) return THC_EWORKSPACE;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PtrArray in;
    MutPtrArray out, rot;
    memset(&in, 0, sizeof in);
    memset(&out, 0, sizeof out);
    memset(&rot, 0, sizeof rot);
    for (uint32_t i = 0; i < n_local; ++i) {
        in.p[i] = grads[i];
        out.p[i] = packed[i];
        if (rotated != nullptr && rotated[i] != nullptr) {
            if (!aligned16(rotated[i])) return THC_EINVAL;
            rot.p[i] = rotated[i];
        }
    }
    TileGeom g = base_geom(ctx, sz, d, round);
    g.worker_base = worker_base;
    const bool bf16 = ctx->cfg.in_dtype == THC_BF16;
    const uint64_t tiles = (sz.d_pad + kTileElems - 1) / kTileElems;
    geom_pass_a(g);
    if (!two_pass) {
        tile_kernel_t kern = bf16 ? pick_tile_kernel<kLoadGradBF16, kStoreQuant>(ctx->cfg.bits, ctx->identity)
                                  : pick_tile_kernel<kLoadGradF32, kStoreQuant>(ctx->cfg.bits, ctx->identity);
        return launch_tile(ctx, kern, g, tiles, n_local, in, out, rot, scales, st);
    }
    PtrArrayP pin;
    MutPtrArrayP pout, prot;
    memcpy(&pin, &in, sizeof pin);
    memcpy(&pout, &out, sizeof pout);
    memcpy(&prot, &rot, sizeof prot);
    pipe_kernel_t kern = bf16 ? pick_pipe_kernel<kCompressBF16>(ctx->cfg.bits, ctx->identity, k)
                              : pick_pipe_kernel<kCompressF32>(ctx->cfg.bits, ctx->identity, k);
    return launch_pipeline(ctx, kern, !bf16, sz, d, n_local, worker_base, round, 1, scales, workspace,
                           pin, pout, prot, st, nullptr, bf16);
}

// Scales and compress in one launch (see thc.h).  Falls back to the two separate calls where
// the fused kernel does not apply.
int thc_prepare_compress(thc_ctx *ctx, const void *const *grads, uint32_t n, uint32_t worker_base,
                         uint64_t d, uint32_t round, float *scales, void *const *packed,
                         float *const *rotated, void *workspace, uint64_t workspace_bytes, void *stream)
{
    int rc = check_launch_ctx(ctx);
    if (rc != THC_OK) return rc;
    thc_sizes_t sz;
    if ((rc = thc_sizes(ctx, d, n, &sz)) != THC_OK) return rc;
    PipePlan pf;
    if (!plan_pipeline_fused(ctx, sz.nblocks, n, &pf)) {
        rc = thc_prepare(ctx, grads, n, d, scales, workspace, workspace_bytes, stream);
        if (rc != THC_OK) return rc;
        return thc_compress(ctx, grads, n, worker_base, d, round, scales, packed, rotated, workspace,
                            workspace_bytes, stream);
    }
    if ((rc = check_ptr_array(grads, n)) != THC_OK) return rc;
    if ((rc = check_ptr_array(packed, n)) != THC_OK) return rc;
    if (scales == nullptr || workspace == nullptr || !aligned16(workspace)) return THC_EINVAL;
    if ((uint64_t)worker_base + n > 0xFFFFFFFFull) return THC_EINVAL;
    if (workspace_bytes < sz.workspace_bytes) return THC_EWORKSPACE;
    PtrArrayP pin;
    MutPtrArrayP pout, prot;
    memset(&pin, 0, sizeof pin);
    memset(&pout, 0, sizeof pout);
    memset(&prot, 0, sizeof prot);
    for (uint32_t i = 0; i < n; ++i) {
        pin.p[i] = grads[i];
        pout.p[i] = packed[i];
        if (rotated != nullptr && rotated[i] != nullptr) {
            if (!aligned16(rotated[i])) return THC_EINVAL;
            prot.p[i] = rotated[i];
        }
    }
    pipe_kernel_t kern = pick_pipe_kernel_kb<kCompressF32Fused, 7>(ctx->cfg.bits, ctx->identity);
    return launch_pipeline(ctx, kern, true, sz, d, n, worker_base, round, 1, scales, workspace, pin, pout,
                           prot, static_cast<cudaStream_t>(stream), scales);
}

int thc_decompress(thc_ctx *ctx, const void *sum, uint32_t divisor, uint64_t d, uint32_t round,
                   const float *scales, float *outp, void *workspace, uint64_t workspace_bytes,
                   void *stream)
{
    int rc = check_launch_ctx(ctx);
    if (rc != THC_OK) return rc;
    thc_sizes_t sz;
    if ((rc = thc_sizes(ctx, d, 1, &sz)) != THC_OK) return rc;
    if (sum == nullptr || outp == nullptr || scales == nullptr || divisor == 0) return THC_EINVAL;
    if (!aligned16(sum) || !aligned16(outp)) return THC_EINVAL;
    const uint32_t k = ctx->cfg.log2_block;
    const bool two_pass = k > (uint32_t)kTileLog2;
    if (two_pass) {
        if (workspace == nullptr || !aligned16(workspace)) return THC_EINVAL;
        if (workspace_bytes < pipeline_workspace_need(ctx, sz.nblocks, sz.nblocks)) return THC_EWORKSPACE;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PtrArray in;
    MutPtrArray out, rot;
    memset(&in, 0, sizeof in);
    memset(&out, 0, sizeof out);
    memset(&rot, 0, sizeof rot);
    in.p[0] = sum;
    out.p[0] = outp;
    TileGeom g = base_geom(ctx, sz, d, round);
    g.divisor = divisor;
    const uint64_t tiles = (sz.d_pad + kTileElems - 1) / kTileElems;
    geom_pass_a(g);
    const uint32_t w = ctx->acc_bits;
    tile_kernel_t k1;
    if (!two_pass) {
        k1 = w == 8 ? pick_tile_kernel<kLoadSum8, kStoreOut>(4, true)
           : w == 16 ? pick_tile_kernel<kLoadSum16, kStoreOut>(4, true)
                     : pick_tile_kernel<kLoadSum32, kStoreOut>(4, true);
        return launch_tile(ctx, k1, g, tiles, 1, in, out, rot, scales, st);
    }
    PtrArrayP pin;
    MutPtrArrayP pout, prot;
    memcpy(&pin, &in, sizeof pin);
    memcpy(&pout, &out, sizeof pout);
    memcpy(&prot, &rot, sizeof prot);
    pipe_kernel_t kern = w == 8 ? pick_pipe_kernel<kDecompress8>(4, true, k)
                       : w == 16 ? pick_pipe_kernel<kDecompress16>(4, true, k)
                                 : pick_pipe_kernel<kDecompress32>(4, true, k);
    return launch_pipeline(ctx, kern, false, sz, d, 1, 0, round, divisor, scales, workspace, pin, pout,
                           prot, st);
}

// thc_aggregate followed by thc_decompress in one launch for the simulated cluster, whose workers'
// packed indices all sit in this GPU's memory (Algorithm 2: the PS line Y = sum_i T[Z_i] feeding
// the worker's estimate line and the inverse RHT): pass A of the inverse transform adds up the
// table values itself, so the sums need not travel through HBM; they are written only on request.
int thc_aggregate_decompress(thc_ctx *ctx, const void *const *packed, uint32_t n, uint64_t d, uint32_t round,
                             const float *scales, float *outp, void *sum_or_null, void *workspace,
                             uint64_t workspace_bytes, void *stream)
{
    int rc = check_launch_ctx(ctx);
    if (rc != THC_OK) return rc;
    if (n == 0 || n > ctx->cfg.workers) return THC_EINVAL;
    thc_sizes_t sz;
    if ((rc = thc_sizes(ctx, d, 1, &sz)) != THC_OK) return rc;
    if ((rc = check_ptr_array(packed, n)) != THC_OK) return rc;
    if (outp == nullptr || scales == nullptr || !aligned16(outp)) return THC_EINVAL;
    if (sum_or_null != nullptr && !aligned16(sum_or_null)) return THC_EINVAL;
    const uint32_t k = ctx->cfg.log2_block;
    if (k <= (uint32_t)kTileLog2 || ctx->cfg.bits != 4 || ctx->cfg.granularity >= 128) {
        // small blocks, and index widths without the byte-lane look-up (there the one launch is
        // slower than the two): the two calls; the sums go to the caller's buffer or to the workspace
        // (without a buffer the sums take the end of the workspace; thc_decompress checks that what
        // is left in front of them is enough for it)
        uint64_t ws_for_decompress = workspace_bytes;
        void *sum = sum_or_null;
        if (sum == nullptr) {
            if (workspace == nullptr || !aligned16(workspace)) return THC_EINVAL;
            const uint64_t room = round_up(sz.sum_bytes, 256);
            if (workspace_bytes < room) return THC_EWORKSPACE;
            ws_for_decompress = (workspace_bytes - room) & ~(uint64_t)255;
            sum = static_cast<unsigned char *>(workspace) + ws_for_decompress;
        }
        if ((rc = thc_aggregate(ctx, packed, n, d, sum, stream)) != THC_OK) return rc;
        return thc_decompress(ctx, sum, n, d, round, scales, outp, workspace, ws_for_decompress, stream);
    }
    if (workspace == nullptr || !aligned16(workspace)) return THC_EINVAL;
    if (workspace_bytes < pipeline_workspace_need(ctx, sz.nblocks, sz.nblocks)) return THC_EWORKSPACE;
    PtrArrayP pin;
    MutPtrArrayP pout, prot;
    memset(&pin, 0, sizeof pin);
    memset(&pout, 0, sizeof pout);
    memset(&prot, 0, sizeof prot);
    for (uint32_t i = 0; i < n; ++i) pin.p[i] = packed[i];
    pout.p[0] = outp;
    pout.p[1] = sum_or_null;
    pipe_kernel_t kern = pick_pipe_kernel<kAggDecompress>(ctx->cfg.bits, true, k);
    return launch_pipeline(ctx, kern, false, sz, d, 1, 0, round, n, scales, workspace, pin, pout, prot,
                           static_cast<cudaStream_t>(stream), nullptr, false, n);
}

int thc_quantize_rotated(thc_ctx *ctx, const float *const *rotated, uint32_t n_local,
                         uint32_t worker_base, uint64_t d, uint32_t round, const float *scales,
                         void *const *packed, void *stream)
{
    int rc = check_launch_ctx(ctx);
    if (rc != THC_OK) return rc;
    thc_sizes_t sz;
    if ((rc = thc_sizes(ctx, d, n_local, &sz)) != THC_OK) return rc;
    if ((rc = check_ptr_array(reinterpret_cast<const void *const *>(rotated), n_local)) != THC_OK) return rc;
    if ((rc = check_ptr_array(packed, n_local)) != THC_OK) return rc;
    if (scales == nullptr) return THC_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PtrArray in;
    MutPtrArray out;
    memset(&in, 0, sizeof in);
    memset(&out, 0, sizeof out);
    for (uint32_t i = 0; i < n_local; ++i) { in.p[i] = rotated[i]; out.p[i] = packed[i]; }
    const uint64_t units = sz.d_pad / 8;
    uint64_t blocks = (units + kThreads - 1) / kThreads;
    const uint64_t cap = (uint64_t)ctx->sm_count * 16;
    if (blocks > cap) blocks = cap;
    const dim3 grid((unsigned)blocks, n_local);
    const uint32_t k = ctx->cfg.log2_block, g = ctx->cfg.granularity;
    const size_t qr_smem = (size_t)(g + 1) * kLutEntryBytes + (size_t)kQrBlockCache * 8;
#define THC_QR(B, I) quantize_rotated_kernel<B, I><<<grid, kThreads, qr_smem, st>>>( \
        in, out, sz.d_pad, k, g, round, worker_base,                         \
        ctx->cfg.range_mode == THC_RANGE_MINMAX ? 1u : 0u, scales, ctx->dev, ctx->keys)
    switch (ctx->cfg.bits) {
    case 1: if (ctx->identity) THC_QR(1, true); else THC_QR(1, false); break;
    case 2: if (ctx->identity) THC_QR(2, true); else THC_QR(2, false); break;
    case 3: if (ctx->identity) THC_QR(3, true); else THC_QR(3, false); break;
    case 4: if (ctx->identity) THC_QR(4, true); else THC_QR(4, false); break;
    default: if (ctx->identity) THC_QR(8, true); else THC_QR(8, false); break;
    }
#undef THC_QR
    THC_CUDA(cudaGetLastError());
    return THC_OK;
}

int thc_aggregate(thc_ctx *ctx, const void *const *packed, uint32_t n, uint64_t d, void *sum,
                  void *stream)
{
    int rc = check_launch_ctx(ctx);
    if (rc != THC_OK) return rc;
    if (n == 0 || n > ctx->cfg.workers) return THC_EINVAL;
    thc_sizes_t sz;
    if ((rc = thc_sizes(ctx, d, n, &sz)) != THC_OK) return rc;
    if ((rc = check_ptr_array(packed, n)) != THC_OK) return rc;
    if (sum == nullptr || !aligned16(sum)) return THC_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PtrArray in;
    memset(&in, 0, sizeof in);
    for (uint32_t i = 0; i < n; ++i) in.p[i] = packed[i];
    const uint64_t units = sz.d_pad / 32;       // the kernel finishes a tail of 8..24 itself
    uint64_t blocks = (units + kThreads - 1) / kThreads;
    if (blocks == 0) blocks = 1;
    const uint64_t cap = (uint64_t)ctx->sm_count * 16;
    if (blocks > cap) blocks = cap;
    unsigned char *s = static_cast<unsigned char *>(sum);
    if (ctx->cfg.bits == 4 && ctx->acc_bits == 8 && ctx->cfg.granularity < 128 && sz.d_pad % 32 == 0) {
        const uint64_t units32 = sz.d_pad / 32;
        uint64_t nb = (units32 + kThreads - 1) / kThreads;
        const uint64_t cap32 = (uint64_t)ctx->sm_count * 64;     // a unit or two per thread: no uneven tail
        if (nb > cap32) nb = cap32;
        aggregate_b4w8_kernel<<<(unsigned)nb, kThreads, 0, st>>>(in, n, units32, ctx->dev,
                                                                  reinterpret_cast<uint4 *>(s));
        THC_CUDA(cudaGetLastError());
        return THC_OK;
    }
    const uint32_t bits = ctx->cfg.bits, g = ctx->cfg.granularity, w = ctx->acc_bits;
    if (bits == 4 && w == 16 && g < 128 && sz.d_pad % 32 == 0) {
        const uint64_t units32 = sz.d_pad / 32;
        uint64_t nb = (units32 + kThreads - 1) / kThreads;
        if (nb > (uint64_t)ctx->sm_count * 64) nb = (uint64_t)ctx->sm_count * 64;
        uint4 *s4 = reinterpret_cast<uint4 *>(s);
        if (g <= 31) aggregate_b4w16_kernel<8><<<(unsigned)nb, kThreads, 0, st>>>(in, n, units32, ctx->dev, s4);
        else if (g <= 63) aggregate_b4w16_kernel<4><<<(unsigned)nb, kThreads, 0, st>>>(in, n, units32, ctx->dev, s4);
        else aggregate_b4w16_kernel<2><<<(unsigned)nb, kThreads, 0, st>>>(in, n, units32, ctx->dev, s4);
        THC_CUDA(cudaGetLastError());
        return THC_OK;
    }
    if ((bits == 1 || (bits == 2 && ctx->identity)) && w == 8 && sz.d_pad % 32 == 0) {
        const uint64_t units32 = sz.d_pad / 32;
        uint64_t nb = (units32 + kThreads - 1) / kThreads;
        if (nb > (uint64_t)ctx->sm_count * 8) nb = (uint64_t)ctx->sm_count * 8;
        if (bits == 1)
            aggregate_small_w8_kernel<1><<<(unsigned)nb, kThreads, 0, st>>>(in, n, units32, g,
                                                                            reinterpret_cast<uint4 *>(s));
        else
            aggregate_small_w8_kernel<2><<<(unsigned)nb, kThreads, 0, st>>>(in, n, units32, 1u,
                                                                            reinterpret_cast<uint4 *>(s));
        THC_CUDA(cudaGetLastError());
        return THC_OK;
    }
    if (bits == 8 && ctx->identity && w == 16 && sz.d_pad % 16 == 0) {
        const uint64_t units16 = sz.d_pad / 16;
        uint64_t nb = (units16 + kThreads - 1) / kThreads;
        if (nb > (uint64_t)ctx->sm_count * 8) nb = (uint64_t)ctx->sm_count * 8;
        aggregate_b8w16_kernel<<<(unsigned)nb, kThreads, 0, st>>>(in, n, units16, reinterpret_cast<uint4 *>(s));
        THC_CUDA(cudaGetLastError());
        return THC_OK;
    }
#define THC_AG(B, W) aggregate_kernel<B, W><<<(unsigned)blocks, kThreads, 0, st>>>(in, n, units, sz.d_pad, ctx->dev, s)
#define THC_AGW(B)                                       \
    do {                                                 \
        if (ctx->acc_bits == 8) THC_AG(B, 8);            \
        else if (ctx->acc_bits == 16) THC_AG(B, 16);     \
        else THC_AG(B, 32);                              \
    } while (0)
    switch (ctx->cfg.bits) {
    case 1: THC_AGW(1); break;
    case 2: THC_AGW(2); break;
    case 3: THC_AGW(3); break;
    case 4: THC_AGW(4); break;
    default: THC_AGW(8); break;
    }
#undef THC_AGW
#undef THC_AG
    THC_CUDA(cudaGetLastError());
    return THC_OK;
}

int thc_error_feedback(thc_ctx *ctx, const void *const *grads, const void *const *packed,
                       uint32_t n_local, uint64_t d, uint32_t round, const float *scales,
                       float *const *ef, void *workspace, uint64_t workspace_bytes, void *stream)
{
    int rc = check_launch_ctx(ctx);
    if (rc != THC_OK) return rc;
    if (ctx->cfg.in_dtype != THC_F32) return THC_EUNSUPPORTED;
    thc_sizes_t sz;
    if ((rc = thc_sizes(ctx, d, 1, &sz)) != THC_OK) return rc;
    if (n_local == 0 || n_local > THC_MAX_WORKERS) return THC_EINVAL;
    if ((rc = check_ptr_array(grads, n_local)) != THC_OK) return rc;
    if ((rc = check_ptr_array(packed, n_local)) != THC_OK) return rc;
    if ((rc = check_ptr_array(reinterpret_cast<const void *const *>(ef), n_local)) != THC_OK) return rc;
    if (scales == nullptr || workspace == nullptr || !aligned16(workspace)) return THC_EINVAL;
    if (workspace_bytes < sz.workspace_bytes) return THC_EWORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (ctx->cfg.log2_block > (uint32_t)kTileLog2) {
        // one launch of the pipeline for all workers: indices in, x_i - RHT^-1(X_i) out
        thc_sizes_t szn;
        if ((rc = thc_sizes(ctx, d, n_local, &szn)) != THC_OK) return rc;
        if (workspace_bytes < szn.workspace_bytes) return THC_EWORKSPACE;
        PtrArrayP pin;
        MutPtrArrayP pout, px;
        memset(&pin, 0, sizeof pin);
        memset(&pout, 0, sizeof pout);
        memset(&px, 0, sizeof px);
        for (uint32_t i = 0; i < n_local; ++i) {
            pin.p[i] = packed[i];
            pout.p[i] = ef[i];
            px.p[i] = const_cast<void *>(grads[i]);
        }
        pipe_kernel_t kern = pick_pipe_kernel<kErrorFeedback>(ctx->cfg.bits, true, ctx->cfg.log2_block);
        return launch_pipeline(ctx, kern, false, szn, d, n_local, 0, round, 1, scales, workspace, pin, pout, px, st);
    }
    const uint64_t ring_bytes = sz.workspace_bytes - round_up(sz.sum_bytes, 256);
    void *values = static_cast<unsigned char *>(workspace) + ring_bytes;
    uint64_t blocks = (d / 4 + kThreads - 1) / kThreads;
    const uint64_t cap = (uint64_t)ctx->sm_count * 16;
    if (blocks > cap) blocks = cap;
    if (blocks == 0) blocks = 1;
    for (uint32_t i = 0; i < n_local; ++i) {
        if ((rc = thc_aggregate(ctx, &packed[i], 1, d, values, stream)) != THC_OK) return rc;
        if ((rc = thc_decompress(ctx, values, 1, d, round, scales, ef[i], workspace, ring_bytes, stream)) != THC_OK)
            return rc;
        ef_subtract_kernel<<<(unsigned)blocks, kThreads, 0, st>>>(static_cast<const float *>(grads[i]), ef[i], d);
        THC_CUDA(cudaGetLastError());
    }
    return THC_OK;
}

int thc_accumulate_error(thc_ctx *ctx, float *const *grads, const float *const *ef, uint32_t n_local,
                         uint64_t d, void *stream)
{
    int rc = check_launch_ctx(ctx);
    if (rc != THC_OK) return rc;
    if (ctx->cfg.in_dtype != THC_F32) return THC_EUNSUPPORTED;
    if (n_local == 0 || n_local > THC_MAX_WORKERS || d == 0) return THC_EINVAL;
    if ((rc = check_ptr_array(reinterpret_cast<const void *const *>(grads), n_local)) != THC_OK) return rc;
    if ((rc = check_ptr_array(reinterpret_cast<const void *const *>(ef), n_local)) != THC_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint64_t blocks = (d / 4 + kThreads - 1) / kThreads;
    const uint64_t cap = (uint64_t)ctx->sm_count * 16;
    if (blocks > cap) blocks = cap;
    if (blocks == 0) blocks = 1;
    for (uint32_t i = 0; i < n_local; ++i) {
        accumulate_kernel<<<(unsigned)blocks, kThreads, 0, st>>>(grads[i], ef[i], d);
        THC_CUDA(cudaGetLastError());
    }
    return THC_OK;
}

int thc_debug_skip_tasks(thc_ctx *ctx, uint32_t count)
{
    int rc = check_launch_ctx(ctx);
    if (rc != THC_OK) return rc;
    THC_CUDA(cudaDeviceSynchronize());
    PipeCounters *pc = reinterpret_cast<PipeCounters *>(ctx->dev->counters);
    THC_CUDA(cudaMemcpy(&pc->head, &count, sizeof count, cudaMemcpyHostToDevice));
    return THC_OK;
}

int thc_status(thc_ctx *ctx, uint32_t *flags, void *stream)
{
    int rc = check_launch_ctx(ctx);
    if (rc != THC_OK) return rc;
    if (flags == nullptr) return THC_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    THC_CUDA(cudaMemcpyAsync(flags, &ctx->dev->status, 4, cudaMemcpyDeviceToHost, st));
    THC_CUDA(cudaMemsetAsync(&ctx->dev->status, 0, 4, st));
    THC_CUDA(cudaStreamSynchronize(st));
    return THC_OK;
}

