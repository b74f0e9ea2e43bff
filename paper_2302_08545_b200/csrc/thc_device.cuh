// Device-side building blocks of libthc: counter RNG, packed-fp32 butterflies, the
// swizzled shared-memory Hadamard rounds and the per-coordinate quantiser.
//
// Arithmetic contract (what makes results reproducible bit for bit):
//   * every fp32 operation is a single IEEE round-to-nearest operation; the file is
//     compiled with -fmad=false, so only the fmaf() calls written here are fused;
//   * the Hadamard transform is radix-2 with stages in ascending stride order and one
//     multiplication by (float)(1/sqrt(B)) at the end (THC paper, Section 5.1: the RHT is
//     (1/sqrt d) H D x; the paper fixes no evaluation order, this is the library's);
//   * random bits come from Philox4x32-10 keyed by the shared seed.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace thc {

constexpr int kTileLog2 = 14;                  // a CTA transforms 2^14 coordinates at a time
constexpr int kTileElems = 1 << kTileLog2;
constexpr int kTileChunks = kTileElems / 4;    // 16-byte chunks
constexpr int kThreads = 256;
constexpr int kSignWordsMax = 1024;            // sign words a tile can need

// Lives in the context's device block.
struct DeviceBlock {
    uint32_t status;             // THC_STATUS_* bits
    uint32_t pad_[31];
    uint32_t counters[5632];     // scheduling counters (self-resetting), 128-byte aligned
    uint4    lut[256];           // by floor(u*g): (-T[z0] as float, 65536/(T[z0+1]-T[z0]), z0, 0)
    uint32_t table[256];         // T
};

struct PhiloxKeys { uint32_t k[20]; };         // the ten round keys, precomputed on the host

// Philox4x32-10 (Salmon et al., SC'11).
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxKeys &keys)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ keys.k[2 * r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ keys.k[2 * r + 1];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Sign diagonal D of the RHT (Section 5.1; "D^r" in Algorithm 3): one Philox call covers
// 128 consecutive padded coordinates, counter = (j/128 lo, j/128 hi, 0xFFFFFFFF, round).
__device__ __forceinline__ uint4 sign_call(uint64_t j, uint32_t round, const PhiloxKeys &keys)
{
    const uint64_t call = j >> 7;
    return philox4x32_10((uint32_t)call, (uint32_t)(call >> 32), 0xFFFFFFFFu, round, keys);
}

// Rounding variates (Section 4.1 needs one uniform per coordinate; Appendix A.2 asks that
// workers draw independently): one call covers 8 consecutive coordinates, 16 bits each,
// counter = (j/8 lo, j/8 hi, worker, round).
__device__ __forceinline__ uint4 round_call(uint64_t j, uint32_t worker, uint32_t round,
                                            const PhiloxKeys &keys)
{
    const uint64_t call = j >> 3;
    return philox4x32_10((uint32_t)call, (uint32_t)(call >> 32), worker, round, keys);
}

// ------------------------------------------------------------------------ clamp range
// Range [lo, hi] of an RHT block (Algorithm 2's m and M).  Norm mode (Section 5.3): the
// scales array holds M per block and m = -M.  Exact mode (Algorithm 1's preliminary stage
// applied to the rotated coordinates): it holds nblocks minima followed by nblocks maxima.
struct BlockRange { float lo, hi; };

__device__ __forceinline__ BlockRange block_range(const float *scales, uint64_t r, uint64_t nblocks,
                                                  uint32_t exact)
{
    BlockRange b;
    if (exact) { b.lo = scales[r]; b.hi = scales[nblocks + r]; }
    else { b.hi = scales[r]; b.lo = -b.hi; }
    return b;
}

// (kappa, offset) of u = sat(fma(r, kappa, offset)): 1/(hi - lo) and -lo/(hi - lo), which for
// lo = -hi are 1/(2M) and exactly 1/2; (0, 0) marks a degenerate block (every index 0).
__device__ __forceinline__ float2 compress_constants(BlockRange b)
{
    if (!(b.hi > b.lo) || !isfinite(b.hi) || !isfinite(b.lo)) return make_float2(0.f, 0.f);
    const double w = (double)b.hi - (double)b.lo;
    return make_float2((float)(1.0 / w), (float)(-(double)b.lo / w));
}

// (step, base) of v = fma(Y, step, base): (hi - lo)/(g * divisor) and lo; (0, 0) for a
// degenerate block (decodes to zeros).  hi == lo (a constant block: every index is 0) gives
// step 0 and base lo: the estimate line of Algorithm 2 with M = m.
__device__ __forceinline__ float2 decode_constants(BlockRange b, uint32_t g, uint32_t divisor)
{
    if (!(b.hi >= b.lo) || !isfinite(b.hi) || !isfinite(b.lo)) return make_float2(0.f, 0.f);
    const double w = (double)b.hi - (double)b.lo;
    return make_float2((float)(w / ((double)g * (double)divisor)), b.lo);
}

// Order-preserving map of fp32 bit patterns onto unsigned integers (for atomic min / max).
__device__ __forceinline__ uint32_t float_key(float f)
{
    const uint32_t u = __float_as_uint(f);
    return u ^ ((u >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k)
{
    return __uint_as_float(k ^ ((k >> 31) ? 0x80000000u : 0xFFFFFFFFu));
}

// ---------------------------------------------------------------- packed fp32 arithmetic
__device__ __forceinline__ float2 add2(float2 a, float2 b) { return __fadd2_rn(a, b); }

// a - b as fma(b, -1, a): one rounding of the exact difference, i.e. the same result as a
// subtraction, expressed with the packed intrinsic so that the compiler keeps operands in
// register pairs.
__device__ __forceinline__ float2 sub2(float2 a, float2 b)
{
    return __ffma2_rn(b, make_float2(-1.0f, -1.0f), a);
}

// One radix-2 butterfly on four independent columns: (a, b) <- (a + b, a - b).
__device__ __forceinline__ void butterfly(float4 &a, float4 &b)
{
    const float2 alo = make_float2(a.x, a.y), ahi = make_float2(a.z, a.w);
    const float2 blo = make_float2(b.x, b.y), bhi = make_float2(b.z, b.w);
    const float2 slo = add2(alo, blo), shi = add2(ahi, bhi);
    const float2 dlo = sub2(alo, blo), dhi = sub2(ahi, bhi);
    a = make_float4(slo.x, slo.y, shi.x, shi.y);
    b = make_float4(dlo.x, dlo.y, dhi.x, dhi.y);
}

// Stages of stride 1 and 2 inside one 16-byte chunk (coordinates 4q .. 4q+3).
__device__ __forceinline__ float4 stages01(float4 v)
{
    const float x = v.x + v.y, y = v.x - v.y, z = v.z + v.w, w = v.z - v.w;
    const float2 s = add2(make_float2(x, y), make_float2(z, w));
    const float2 d = sub2(make_float2(x, y), make_float2(z, w));
    return make_float4(s.x, s.y, d.x, d.y);
}

__device__ __forceinline__ float4 scale4(float4 v, float c)
{
    const float2 c2 = make_float2(c, c);
    const float2 lo = __fmul2_rn(make_float2(v.x, v.y), c2);
    const float2 hi = __fmul2_rn(make_float2(v.z, v.w), c2);
    return make_float4(lo.x, lo.y, hi.x, hi.y);
}

// Flip the signs of a chunk by bits [0,4) of `bits` (bit e set -> element e negated).
__device__ __forceinline__ float4 flip4(float4 v, uint32_t bits)
{
    v.x = __uint_as_float(__float_as_uint(v.x) ^ ((bits << 31) & 0x80000000u));
    v.y = __uint_as_float(__float_as_uint(v.y) ^ ((bits << 30) & 0x80000000u));
    v.z = __uint_as_float(__float_as_uint(v.z) ^ ((bits << 29) & 0x80000000u));
    v.w = __uint_as_float(__float_as_uint(v.w) ^ ((bits << 28) & 0x80000000u));
    return v;
}

// ------------------------------------------------------------------- shared-memory tile
// The tile holds 4096 chunks.  Chunk c is stored at c ^ ((c >> 4) & 7): with this XOR every
// access pattern below (consecutive chunks per lane, or one chunk per lane at any
// power-of-two stride) touches eight distinct 16-byte bank groups per quarter warp.
__device__ __forceinline__ int swz(int c) { return c ^ ((c >> 4) & 7); }

// Butterfly stages on chunk-index bits [sp, sp+E) of the tile, ascending.  Each thread owns
// whole groups of 2^E chunks, so the update is in place; callers separate rounds by a
// block barrier.
template <int E>
__device__ __forceinline__ void fwht_round(float4 *tile, int sp, int tid)
{
    constexpr int N = 1 << E;
    constexpr int kGroups = kTileChunks >> E;
#pragma unroll 1
    for (int G = tid; G < kGroups; G += kThreads) {
        const int low = G & ((1 << sp) - 1);
        const int base = ((G >> sp) << (sp + E)) | low;
        float4 v[N];
#pragma unroll
        for (int m = 0; m < N; ++m) v[m] = tile[swz(base + (m << sp))];
#pragma unroll
        for (int t = 0; t < E; ++t) {
#pragma unroll
            for (int m = 0; m < N; ++m) {
                if (!(m & (1 << t))) butterfly(v[m], v[m | (1 << t)]);
            }
        }
#pragma unroll
        for (int m = 0; m < N; ++m) tile[swz(base + (m << sp))] = v[m];
    }
}

// All stages on chunk bits [lo, hi), in rounds of at most four bits.
__device__ __forceinline__ void fwht_rounds(float4 *tile, int lo, int hi, int tid)
{
    int sp = lo;
    while (sp < hi) {
        const int e = min(4, hi - sp);
        switch (e) {
        case 4: fwht_round<4>(tile, sp, tid); break;
        case 3: fwht_round<3>(tile, sp, tid); break;
        case 2: fwht_round<2>(tile, sp, tid); break;
        default: fwht_round<1>(tile, sp, tid); break;
        }
        sp += e;
        __syncthreads();
    }
}

// --------------------------------------------------------------------------- quantiser
// The quantiser's table in shared memory, indexed by f = floor(u g): what the rounding rule
// needs about the table interval [T[z0], T[z0+1]] that holds f.  Consecutive entries are 128
// bytes apart and every entry is replicated over lanes so that a warp's look-ups (random f per
// lane) never meet in a bank:
//   indices of up to 4 bits   16 copies of 8 bytes   (R16 = 65536 / gap as fp32,
//                                                     bf16(-T[z0]) << 16 | z0: table values up to
//                                                     255 are exact in bf16)
//   8-bit indices              8 copies of 16 bytes  (-T[z0] as fp32, R16, z0, 0)
constexpr int kLutEntryBytes = 128;

template <int BITS, bool IDENTITY>
struct LutKind { static constexpr bool k8 = !IDENTITY && BITS <= 4; };

template <bool LUT8>
__device__ __forceinline__ void lut_fill(unsigned char *lut, const DeviceBlock *dev, uint32_t g, int tid, int nthreads)
{
    if (LUT8) {
        for (int idx = tid; idx < (int)(g + 1) * 16; idx += nthreads) {
            const uint4 e = dev->lut[idx / 16];
            reinterpret_cast<uint2 *>(lut)[idx] = make_uint2(e.y, (e.x & 0xFFFF0000u) | e.z);
        }
    } else {
        for (int idx = tid; idx < (int)(g + 1) * 8; idx += nthreads)
            reinterpret_cast<uint4 *>(lut)[idx] = dev->lut[idx / 8];
    }
}

// Shared-space byte address of this lane's copy of entry 0, minus 0x4B000000 * 128: the bits of
// the float 2^23 + f, times 128, plus this value is the address of entry f.
template <bool LUT8>
__device__ __forceinline__ uint32_t lut_lane_addr(const unsigned char *lut, int lane)
{
    const uint32_t copy = LUT8 ? (uint32_t)(lane & 15) * 8u : (uint32_t)(lane & 7) * 16u;
    return (uint32_t)__cvta_generic_to_shared(lut) + copy - 0x4B000000u * (uint32_t)kLutEntryBytes;
}

// Stochastic quantisation of eight consecutive rotated coordinates to table indices
// (Algorithm 2, worker lines; Section 4.1 for the rounding rule):
//   u = sat(fma(r, kappa, offset))          position in [m, M] on the unit interval, truncated
//   f = floor(u * g)                         (one round-down fma onto 2^23; exact)
//   z0 = index of the table value at or below u*g, delta = fma(u, g, -T[z0])
//   up iff u16 < RN(2^16 delta / gap)        (one fma onto 2^23, integer compare)
// kappa = 1/(2M) and offset = 1/2; kappa = offset = 0 encodes a degenerate block (index 0).
// `lut_addr` comes from lut_lane_addr (unused for the identity table).  Returns the indices
// packed BITS apiece, coordinate 0 in the low bits.
template <int BITS, bool IDENTITY>
__device__ __forceinline__ uint64_t quantize8(const float (&r)[8], float kappa, float offset,
                                              float gf, uint4 rnd, uint32_t lut_addr)
{
    constexpr bool kLut8 = LutKind<BITS, IDENTITY>::k8;
    const uint32_t words[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
    // Indices are accumulated as z * 2^(BITS*slot) with multiply-adds into two 32-bit halves
    // (coordinates 0-3 and 4-7).  With the 8-byte entries the whole second word is multiplied
    // in: what its upper half leaves above bit 16 is cut off at the end (4 BITS <= 16 valid bits).
    uint32_t acc[2] = {0u, 0u};
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        float u;
        asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(u) : "f"(r[e]), "f"(kappa), "f"(offset));
        const float t = __fmaf_rd(u, gf, 8388608.0f);          // 2^23 + floor(u * g)
        // bits of 2^23 + u16
        const uint32_t ub = (e & 1) ? __byte_perm(words[e >> 1], 0x4B000000u, 0x7432)
                                    : __byte_perm(words[e >> 1], 0x4B000000u, 0x7410);
        uint32_t zw;
        float tau;
        if (IDENTITY) {
            zw = __float_as_uint(t) & 0xFFu;
            const float delta = fmaf(u, gf, 8388608.0f - t);
            tau = fmaf(delta, 65536.0f, 8388608.0f);
        } else if (kLut8) {
            const uint32_t a = __float_as_uint(t) * (uint32_t)kLutEntryBytes + lut_addr;
            uint32_t x, y;
            asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(x), "=r"(y) : "r"(a));
            const float delta = fmaf(u, gf, __uint_as_float(y & 0xFFFF0000u));
            tau = fmaf(delta, __uint_as_float(x), 8388608.0f);
            zw = y;
        } else {
            const uint32_t a = __float_as_uint(t) * (uint32_t)kLutEntryBytes + lut_addr;
            uint32_t x, y, z, w;
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(x), "=r"(y), "=r"(z), "=r"(w) : "r"(a));
            const float delta = fmaf(u, gf, __uint_as_float(x));
            tau = fmaf(delta, __uint_as_float(y), 8388608.0f);
            zw = z;
        }
        const int h = e >> 2;
        const uint32_t weight = 1u << (BITS * (e & 3));
        acc[h] = zw * weight + acc[h];
        if (ub < __float_as_uint(tau)) acc[h] += weight;
    }
    if constexpr (BITS == 8) return (uint64_t)acc[0] | ((uint64_t)acc[1] << 32);
    if constexpr (BITS == 4) return (uint64_t)__byte_perm(acc[0], acc[1], 0x5410);
    constexpr uint32_t mask = (1u << (4 * BITS)) - 1u;
    return (uint64_t)((acc[0] & mask) | ((acc[1] & mask) << (4 * BITS)));
}

}  // namespace thc
