// Device-side building blocks: 32-byte tile loads, the counter-based random
// bits, and the per-tile bodies of the three O(n) passes (statistics, stochastic
// pruning, FP quantisation + packing).
//
// One tile = kTileElems consecutive elements handled by one CTA of kThreads
// threads.  In every load step thread t takes the t-th 32-byte chunk of a
// kThreads*32-byte span (one 256-bit load), so a warp instruction touches 1 KiB
// of contiguous memory.  A chunk holds kChunk = 8 (fp32) or 16 (bf16) elements
// and always starts at an element index that is a multiple of 8: the eight
// elements that share one block of random bits stay in one thread.
#pragma once

#include <cstdint>
#include <cstring>
#include <cuda_runtime.h>

#include "lgn.h"

namespace lgn {

// Launch shape; the defaults are the measured optimum, the macros exist for sweeps.
#ifndef LGN_THREADS
#define LGN_THREADS 256
#endif
#ifndef LGN_TILE_ELEMS
#define LGN_TILE_ELEMS 32768
#endif
#ifndef LGN_MIN_CTAS
#define LGN_MIN_CTAS 4
#endif
#ifndef LGN_LOADS_IN_FLIGHT
#define LGN_LOADS_IN_FLIGHT 4
#endif
constexpr int kThreads   = LGN_THREADS;
constexpr int kWarps     = kThreads / 32;
constexpr int kTileElems = LGN_TILE_ELEMS;
constexpr int kMinCtas   = LGN_MIN_CTAS;      // resident CTAs per SM the kernels are compiled for
constexpr int kInFlight  = LGN_LOADS_IN_FLIGHT;   // 32-byte loads a thread issues before it uses the first
#ifndef LGN_PREFETCH_STEPS
#define LGN_PREFETCH_STEPS 4
#endif
// Load steps of a whole tile that are requested into L2 ahead of the register loads (0: none).  A
// thread holds only one or two 32-byte loads in registers; the lines of the next few steps are
// asked for with prefetch.global.L2 (no register, no wait), so that the register load that
// follows finds them in L2.  Four steps (32 KiB per CTA) is the measured optimum.
constexpr int kPrefetchSteps = LGN_PREFETCH_STEPS;

template <int DT> struct ElemTraits;
template <> struct ElemTraits<LGN_F32>  { static constexpr int kChunk = 8;  static constexpr int kBytes = 4; };
template <> struct ElemTraits<LGN_BF16> { static constexpr int kChunk = 16; static constexpr int kBytes = 2; };

__device__ __forceinline__ float    u2f(uint32_t u) { return __uint_as_float(u); }
__device__ __forceinline__ uint32_t f2u(float f)    { return __float_as_uint(f); }

struct Chunk { uint32_t w[8]; };          // 32 bytes

// ---------------------------------------------------------------- loads / stores
enum class Ld { Keep, Stream };   // Keep: normal L2 policy (the tensor is read again); Stream: evict first

// WIDE: one 256-bit access.  The out-of-line general tile bodies use two 128-bit
// accesses instead (the 256-bit form is kept to code inlined into a kernel).
template <Ld P, bool WIDE>
__device__ __forceinline__ Chunk ld32(const void *p) {
    Chunk c;
    if (WIDE) {
        if (P == Ld::Keep)
            asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(c.w[0]), "=r"(c.w[1]), "=r"(c.w[2]), "=r"(c.w[3]),
                           "=r"(c.w[4]), "=r"(c.w[5]), "=r"(c.w[6]), "=r"(c.w[7]) : "l"(p));
        else
            asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(c.w[0]), "=r"(c.w[1]), "=r"(c.w[2]), "=r"(c.w[3]),
                           "=r"(c.w[4]), "=r"(c.w[5]), "=r"(c.w[6]), "=r"(c.w[7]) : "l"(p));
    } else {
        asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(c.w[0]), "=r"(c.w[1]), "=r"(c.w[2]), "=r"(c.w[3]) : "l"(p));
        asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4+16];"
                     : "=r"(c.w[4]), "=r"(c.w[5]), "=r"(c.w[6]), "=r"(c.w[7]) : "l"(p));
    }
    return c;
}

template <bool WIDE>
__device__ __forceinline__ void st32_stream(void *p, const Chunk &c) {
    if (WIDE) {
        asm volatile("st.global.L1::no_allocate.L2::evict_first.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                     :: "l"(p), "r"(c.w[0]), "r"(c.w[1]), "r"(c.w[2]), "r"(c.w[3]),
                        "r"(c.w[4]), "r"(c.w[5]), "r"(c.w[6]), "r"(c.w[7]) : "memory");
    } else {
        asm volatile("st.global.cs.v4.b32 [%0], {%1,%2,%3,%4};"
                     :: "l"(p), "r"(c.w[0]), "r"(c.w[1]), "r"(c.w[2]), "r"(c.w[3]) : "memory");
        asm volatile("st.global.cs.v4.b32 [%0+16], {%1,%2,%3,%4};"
                     :: "l"(p), "r"(c.w[4]), "r"(c.w[5]), "r"(c.w[6]), "r"(c.w[7]) : "memory");
    }
}

__device__ __forceinline__ void st4_stream(void *p, uint32_t v) {
    asm volatile("st.global.cs.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

// The chunk that starts at element index i (a multiple of kChunk).  FULL: the
// whole chunk lies inside [0, n); otherwise elements at or past n read as zero.
template <int DT, bool FULL, Ld P>
__device__ __forceinline__ Chunk load_chunk(const void *g, uint64_t i, uint64_t n) {
    constexpr int C = ElemTraits<DT>::kChunk;
    if constexpr (FULL) return ld32<P, true>(static_cast<const char *>(g) + i * ElemTraits<DT>::kBytes);
    if (i + C <= n) return ld32<P, false>(static_cast<const char *>(g) + i * ElemTraits<DT>::kBytes);
    Chunk c;
    #pragma unroll
    for (int k = 0; k < 8; ++k) c.w[k] = 0u;
    if (DT == LGN_F32) {
        const uint32_t *p = static_cast<const uint32_t *>(g);
        #pragma unroll
        for (int k = 0; k < 8; ++k) if (i + k < n) c.w[k] = p[i + k];
    } else {
        const uint16_t *p = static_cast<const uint16_t *>(g);
        #pragma unroll
        for (int k = 0; k < 16; ++k) if (i + k < n) c.w[k >> 1] |= (uint32_t)p[i + k] << ((k & 1) * 16);
    }
    return c;
}

// Store a chunk of output elements of the tensor's own type at element index i;
// elements at or past n are not written.
template <int DT, bool FULL>
__device__ __forceinline__ void store_chunk(void *out, uint64_t i, uint64_t n, const Chunk &c) {
    constexpr int C = ElemTraits<DT>::kChunk;
    if (FULL || i + C <= n) {
        st32_stream<FULL>(static_cast<char *>(out) + i * ElemTraits<DT>::kBytes, c);
        return;
    }
    if (DT == LGN_F32) {
        uint32_t *p = static_cast<uint32_t *>(out);
        #pragma unroll
        for (int k = 0; k < 8; ++k) if (i + k < n) p[i + k] = c.w[k];
    } else {
        uint16_t *p = static_cast<uint16_t *>(out);
        #pragma unroll
        for (int k = 0; k < 16; ++k) if (i + k < n) p[i + k] = (uint16_t)(c.w[k >> 1] >> ((k & 1) * 16));
    }
}

// fp32 bit pattern of element k of a chunk (bf16 widened exactly).
template <int DT>
__device__ __forceinline__ uint32_t elem_bits(const Chunk &c, int k) {
    if (DT == LGN_F32) return c.w[k];
    return (k & 1) ? (c.w[k >> 1] & 0xFFFF0000u) : (c.w[k >> 1] << 16);
}

// Software-pipelined walk over a tile's load steps: two register buffers of
// kGroup chunks each; the loads of the next group are issued before the current
// group is processed, so a thread always has loads in flight while it computes.
// body(buf, j) processes the kGroup chunks of load steps j .. j+kGroup-1.
template <int DT, bool FULL, Ld P, int kLoads, int kGroup, class Body>
__device__ __forceinline__ void pipelined_tile(const void *g, uint64_t tile_base, uint64_t n, Body body) {
    constexpr int C = ElemTraits<DT>::kChunk;
    static_assert(kLoads % (2 * kGroup) == 0, "load steps come in pairs of groups");
    Chunk a[kGroup], b[kGroup];
    // this thread's chunk of load step 0; step j lies j * kStepBytes further on
    const char *mine = static_cast<const char *>(g) + (tile_base + (uint64_t)threadIdx.x * C) * ElemTraits<DT>::kBytes;
    constexpr int kStepBytes = kThreads * 32;
    if (FULL && kPrefetchSteps > 0) {
        #pragma unroll
        for (int j = kGroup; j < kGroup + kPrefetchSteps && j < kLoads; ++j)
            asm volatile("prefetch.global.L2 [%0];" :: "l"(mine + (size_t)j * kStepBytes));
    }
    #pragma unroll
    for (int j = 0; j < kGroup; ++j)
        a[j] = load_chunk<DT, FULL, P>(g, tile_base + (uint64_t)(j * kThreads + threadIdx.x) * C, n);
    #pragma unroll 1
    for (int j0 = 0; j0 < kLoads; j0 += 2 * kGroup) {
        if (FULL && kPrefetchSteps > 0) {
            #pragma unroll
            for (int j = 0; j < 2 * kGroup; ++j)
                if (j0 + kGroup + kPrefetchSteps + j < kLoads)
                    asm volatile("prefetch.global.L2 [%0];" :: "l"(mine + (size_t)(j0 + kGroup + kPrefetchSteps + j) * kStepBytes));
        }
        #pragma unroll
        for (int j = 0; j < kGroup; ++j)
            b[j] = load_chunk<DT, FULL, P>(g, tile_base + (uint64_t)((j0 + kGroup + j) * kThreads + threadIdx.x) * C, n);
        body(a, j0);
        if (j0 + 2 * kGroup < kLoads) {
            #pragma unroll
            for (int j = 0; j < kGroup; ++j)
                a[j] = load_chunk<DT, FULL, P>(g, tile_base + (uint64_t)((j0 + 2 * kGroup + j) * kThreads + threadIdx.x) * C, n);
        }
        body(b, j0 + kGroup);
    }
}

// ---------------------------------------------------------------- random bits
// Philox4x32 (Salmon et al., SC'11), seven rounds: each round is two 32x32->64
// multiplies with the halves crossed and xored with the counter and a
// Weyl-stepped key.  One block serves eight consecutive elements, 16 bits each:
// element 8b + e takes word e/2, low half if e is even, high half if odd.
constexpr int kPhiloxRounds = 7;

// The two Weyl increments of the key schedule.  They are handed to the kernels
// as run-time values (not literals) so that round r's key is formed as
// key + r*W by the multiply-add pipe instead of by a chain of integer adds on
// the busier ALU pipe.
struct Weyl { uint32_t w0, w1; };
constexpr uint32_t kWeyl0 = 0x9E3779B9u, kWeyl1 = 0xBB67AE85u;

__device__ __forceinline__ uint4 rand_block(uint64_t seed, uint64_t b, const Weyl &wy) {
    uint32_t c0 = (uint32_t)b, c1 = (uint32_t)(b >> 32), c2 = 0u, c3 = 0u;
    const uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    #pragma unroll
    for (int r = 0; r < kPhiloxRounds; ++r) {
        const unsigned long long p0 = (unsigned long long)0xD2511F53u * c0;
        const unsigned long long p1 = (unsigned long long)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ (k0 + (uint32_t)r * wy.w0);
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ (k1 + (uint32_t)r * wy.w1);
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Blocks b and b + 1 for an even b (the 16 elements of a bf16 chunk), rounds interleaved so
// that each round key is formed once for both.
__device__ __forceinline__ void rand_block2(uint64_t seed, uint64_t b, const Weyl &wy, uint4 &ra, uint4 &rb) {
    uint32_t a0 = (uint32_t)b, a1 = (uint32_t)(b >> 32), a2 = 0u, a3 = 0u;
    uint32_t b0 = a0 + 1u, b1 = a1, b2 = 0u, b3 = 0u;       // b is even: no carry into the second word
    const uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    #pragma unroll
    for (int r = 0; r < kPhiloxRounds; ++r) {
        const uint32_t key0 = k0 + (uint32_t)r * wy.w0, key1 = k1 + (uint32_t)r * wy.w1;
        const unsigned long long p0 = (unsigned long long)0xD2511F53u * a0, p1 = (unsigned long long)0xCD9E8D57u * a2;
        const unsigned long long q0 = (unsigned long long)0xD2511F53u * b0, q1 = (unsigned long long)0xCD9E8D57u * b2;
        const uint32_t na0 = (uint32_t)(p1 >> 32) ^ a1 ^ key0, na2 = (uint32_t)(p0 >> 32) ^ a3 ^ key1;
        const uint32_t nb0 = (uint32_t)(q1 >> 32) ^ b1 ^ key0, nb2 = (uint32_t)(q0 >> 32) ^ b3 ^ key1;
        a1 = (uint32_t)p1; a3 = (uint32_t)p0; a0 = na0; a2 = na2;
        b1 = (uint32_t)q1; b3 = (uint32_t)q0; b0 = nb0; b2 = nb2;
    }
    ra = make_uint4(a0, a1, a2, a3);
    rb = make_uint4(b0, b1, b2, b3);
}

// The C/8 blocks of the chunk that starts at element i.
template <int DT, bool FULL>
__device__ __forceinline__ void rand_chunk(uint64_t seed, uint64_t i, const Weyl &wy, uint4 (&rr)[ElemTraits<DT>::kChunk / 8]) {
    if constexpr (DT == LGN_BF16 && FULL) {
        rand_block2(seed, i >> 3, wy, rr[0], rr[1]);
    } else {
        #pragma unroll
        for (int b = 0; b < ElemTraits<DT>::kChunk / 8; ++b) rr[b] = rand_block(seed, (i >> 3) + b, wy);
    }
}

__device__ __forceinline__ uint32_t rand_word(const uint4 &r, int e) {
    return (e >> 1) == 0 ? r.x : (e >> 1) == 1 ? r.y : (e >> 1) == 2 ? r.z : r.w;
}

// The element's 16 random bits as an integer and as a float (the conversion of a
// 16-bit half of a register is one instruction on the otherwise idle
// conversion unit).
__device__ __forceinline__ uint32_t rand_h(const uint4 &r, int e) {
    const uint32_t w = rand_word(r, e);
    return (e & 1) ? (w >> 16) : (w & 0xFFFFu);
}
__device__ __forceinline__ float rand_hf(const uint4 &r, int e) {
    const uint32_t w = rand_word(r, e);
    return (e & 1) ? (float)(unsigned short)(w >> 16) : (float)(unsigned short)(w & 0xFFFFu);
}
// eps = (h + 1) / 2^16 in (0,1]: exact in fp32.
__device__ __forceinline__ float eps_of(const uint4 &r, int e) {
    return fmaf(rand_hf(r, e), 0x1p-16f, 0x1p-16f);
}

// ---------------------------------------------------------------- statistics
// log2 of a magnitude scaled by 2^24.  The scaling (an exact multiply) lifts
// every fp32 subnormal into the normal range, so the single-instruction
// flush-to-zero form of the hardware approximation can be used: zero gives -inf,
// everything else log2|x| + 24.  Magnitudes must stay below 2^104 (the product
// must not overflow).
constexpr float kLogShift = 24.0f;
__device__ __forceinline__ float lg2_scaled(float a) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(a * 16777216.0f));
    return y;
}

struct StatsAcc {            // per thread, in log2 units
    double s1 = 0.0, s2 = 0.0;
    unsigned long long cnt = 0;
    unsigned long long right = 0;   // extended pass only: entries of the right mode (mask byte != 0)
    float amax = 0.f;               // extended pass only: largest magnitude of the whole tensor
};

// Adds one tile to the thread's accumulators.  y = log2|x| + 24 in fp32.  The sums
// are taken of d = y - P, where the pivot P is the largest y in the first run
// of this thread's elements that holds a nonzero: d stays of the order of the
// spread of the data whatever its scale, so short fp32 runs of d and d^2 lose
// nothing that matters, and a tensor whose magnitudes are all equal gives a
// variance of exactly zero.  Runs go to fp64 accumulators; the pivot is taken
// out again in fp64 at the end of the tile:
//   sum y = sum d + c P,   sum y^2 = sum d^2 + 2 P sum d + c P^2.
template <int DT, bool FULL, int TILE = kTileElems>
__device__ __forceinline__ void stats_tile(const void *g, uint64_t tile_base, uint64_t n, StatsAcc &acc) {
    constexpr int C = ElemTraits<DT>::kChunk;
    constexpr int kLoads = TILE / (kThreads * C);   // 8 (fp32) or 4 (bf16)
    constexpr int kGroup = 16 / C;                        // chunks per register buffer (two buffers): one run of 16
    const float kUnset = -__int_as_float(0x7F800000);     // -inf: no nonzero seen yet
    float P = kUnset;
    if constexpr (FULL && DT == LGN_BF16) {
        // Whole bf16 tiles (the pass is bound by instruction issue there; on fp32 tiles, which wait
        // for memory, this form measured 1 % slower): the thread's 128 (or 256) pivoted terms of
        // the tile are summed in fp32 (they are of the order of the spread, a sum of squares stays
        // far below 2^24 ulps) and go to fp64 once per tile; the pivot is fixed by the first group
        // of 16 that holds a nonzero.
        float s1 = 0.f, s2 = 0.f, cf = 0.f;
        pipelined_tile<DT, FULL, Ld::Keep, kLoads, kGroup>(g, tile_base, n, [&](const Chunk (&v)[kGroup], int) {
            float y[kGroup * C];
            #pragma unroll
            for (int idx = 0; idx < kGroup * C; ++idx)
                y[idx] = lg2_scaled(fabsf(u2f(elem_bits<DT>(v[idx / C], idx % C))));      // -inf for zero
            if (P == kUnset) {
                #pragma unroll
                for (int idx = 0; idx < kGroup * C; ++idx) P = fmaxf(P, y[idx]);
            }
            #pragma unroll
            for (int idx = 0; idx < kGroup * C; ++idx) {
                if (y[idx] != kUnset) {                    // predicated: no select, no integer add
                    const float d = y[idx] - P;
                    s1 += d;
                    s2 = fmaf(d, d, s2);
                    cf += 1.0f;                            // exact: at most 256 per tile
                }
            }
        });
        if (cf != 0.f) {
            const double p = (double)P - (double)kLogShift, c = (double)cf, D1 = (double)s1, D2 = (double)s2;
            acc.s1 += D1 + c * p;
            acc.s2 += D2 + p * (2.0 * D1 + c * p);
            acc.cnt += (unsigned long long)cf;
        }
        return;
    }
    double D1 = 0.0, D2 = 0.0;
    unsigned long long Cn = 0;
    pipelined_tile<DT, FULL, Ld::Keep, kLoads, kGroup>(g, tile_base, n, [&](const Chunk (&v)[kGroup], int) {
        #pragma unroll
        for (int r = 0; r < kGroup * C / 16; ++r) {       // runs of 16 elements
            float y[16];
            #pragma unroll
            for (int e = 0; e < 16; ++e) {
                const int idx = r * 16 + e;
                y[e] = lg2_scaled(fabsf(u2f(elem_bits<DT>(v[idx / C], idx % C))));   // -inf for zero
            }
            if (P == kUnset) {
                #pragma unroll
                for (int e = 0; e < 16; ++e) P = fmaxf(P, y[e]);
            }
            float s1 = 0.f, s2 = 0.f, cf = 0.f;            // cf: nonzeros of this run, exact in fp32
            #pragma unroll
            for (int e = 0; e < 16; ++e) {
                if (y[e] != kUnset) {                      // predicated: no select, no integer add
                    const float d = y[e] - P;
                    s1 += d;
                    s2 = fmaf(d, d, s2);
                    cf += 1.0f;
                }
            }
            const uint32_t c = (uint32_t)cf;
            D1 += (double)s1;
            D2 += (double)s2;
            Cn += c;
        }
    });
    if (Cn) {
        const double p = (double)P - (double)kLogShift, c = (double)Cn;   // pivot in true log2 units
        acc.s1 += D1 + c * p;
        acc.s2 += D2 + p * (2.0 * D1 + c * p);
        acc.cnt += Cn;
    }
}

// The extended statistics tile: what stats_tile computes, restricted to the
// entries whose byte in `mask` is non-zero when MASKED (the right mode of a
// bi-modal gradient; the appendix's steps 1 and 3), plus the number of such
// entries and the largest magnitude of the whole tile (Algorithm 1's max|X|).
// Same pivoted sums as stats_tile.  Serves whole and ragged tiles; one chunk per
// load step with the next step's loads issued before the current one is used.
// The mask bytes of a chunk are the C bytes at the chunk's element index.
template <int DT>
__device__ __forceinline__ void load_mask_chunk(const uint8_t *mask, uint64_t i, uint64_t n, uint32_t (&m)[4]) {
    constexpr int C = ElemTraits<DT>::kChunk;
    m[0] = m[1] = m[2] = m[3] = 0u;
    if (i + C <= n) {
        if (C == 8) { const uint2 v = __ldg(reinterpret_cast<const uint2 *>(mask + i)); m[0] = v.x; m[1] = v.y; }
        else        { const uint4 v = __ldg(reinterpret_cast<const uint4 *>(mask + i)); m[0] = v.x; m[1] = v.y; m[2] = v.z; m[3] = v.w; }
    } else {
        #pragma unroll
        for (int k = 0; k < C; ++k) if (i + k < n) m[k >> 2] |= (uint32_t)mask[i + k] << ((k & 3) * 8);
    }
}

template <int DT, bool MASKED, int TILE = kTileElems>
__device__ __forceinline__ void stats_tile_ext(const void *g, const uint8_t *mask, uint64_t tile_base, uint64_t n,
                                               StatsAcc &acc) {
    constexpr int C = ElemTraits<DT>::kChunk;
    constexpr int kLoads = TILE / (kThreads * C);
    const float kUnset = -__int_as_float(0x7F800000);
    float P = kUnset, amax = 0.f;
    double D1 = 0.0, D2 = 0.0;
    unsigned long long Cn = 0, Rn = 0;
    auto at = [&](int j) { return tile_base + (uint64_t)(j * kThreads + threadIdx.x) * C; };
    Chunk cur = load_chunk<DT, false, Ld::Keep>(g, at(0), n), nxt = cur;
    uint32_t mcur[4] = {~0u, ~0u, ~0u, ~0u}, mnxt[4] = {~0u, ~0u, ~0u, ~0u};
    if (MASKED) load_mask_chunk<DT>(mask, at(0), n, mcur);
    #pragma unroll 1
    for (int j = 0; j < kLoads; ++j) {
        if (j + 1 < kLoads) {
            nxt = load_chunk<DT, false, Ld::Keep>(g, at(j + 1), n);
            if (MASKED) load_mask_chunk<DT>(mask, at(j + 1), n, mnxt);
        }
        float y[C];
        bool in[C];
        #pragma unroll
        for (int e = 0; e < C; ++e) {
            const float a = fabsf(u2f(elem_bits<DT>(cur, e)));
            amax = fmaxf(amax, a);
            y[e] = lg2_scaled(a);
            const bool right = !MASKED || ((mcur[e >> 2] >> ((e & 3) * 8)) & 0xFFu) != 0u;
            if (MASKED) Rn += right ? 1u : 0u;
            in[e] = right && y[e] != kUnset;
        }
        if (P == kUnset) {
            #pragma unroll
            for (int e = 0; e < C; ++e) if (in[e]) P = fmaxf(P, y[e]);
        }
        float s1 = 0.f, s2 = 0.f, cf = 0.f;
        #pragma unroll
        for (int e = 0; e < C; ++e) {
            if (in[e]) {
                const float d = y[e] - P;
                s1 += d;
                s2 = fmaf(d, d, s2);
                cf += 1.0f;
            }
        }
        D1 += (double)s1;
        D2 += (double)s2;
        Cn += (uint32_t)cf;
        cur = nxt;
        #pragma unroll
        for (int k = 0; k < 4; ++k) mcur[k] = mnxt[k];
    }
    if (Cn) {
        const double p = (double)P - (double)kLogShift, c = (double)Cn;
        acc.s1 += D1 + c * p;
        acc.s2 += D2 + p * (2.0 * D1 + c * p);
        acc.cnt += Cn;
    }
    acc.right += Rn;
    acc.amax = fmaxf(acc.amax, amax);
}

// Fixed-shape tree over the CTA; the result is valid in thread 0.
__device__ __forceinline__ void warp_reduce(StatsAcc &acc, int width) {
    for (int off = width / 2; off > 0; off >>= 1) {
        acc.s1 += __shfl_down_sync(0xFFFFFFFFu, acc.s1, off);
        acc.s2 += __shfl_down_sync(0xFFFFFFFFu, acc.s2, off);
        acc.cnt += __shfl_down_sync(0xFFFFFFFFu, acc.cnt, off);
        acc.right += __shfl_down_sync(0xFFFFFFFFu, acc.right, off);
        acc.amax = fmaxf(acc.amax, __shfl_down_sync(0xFFFFFFFFu, acc.amax, off));
    }
}

__device__ __forceinline__ void block_reduce(StatsAcc &acc, double *sm /* 5*kWarps */) {
    warp_reduce(acc, 32);
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    __syncthreads();                      // sm may still be in use by an earlier reduction
    if (l == 0) {
        sm[w] = acc.s1; sm[kWarps + w] = acc.s2; sm[2 * kWarps + w] = __longlong_as_double((long long)acc.cnt);
        sm[3 * kWarps + w] = __longlong_as_double((long long)acc.right); sm[4 * kWarps + w] = (double)acc.amax;
    }
    __syncthreads();
    if (w == 0) {
        StatsAcc t;
        if (l < kWarps) {
            t.s1 = sm[l]; t.s2 = sm[kWarps + l]; t.cnt = (unsigned long long)__double_as_longlong(sm[2 * kWarps + l]);
            t.right = (unsigned long long)__double_as_longlong(sm[3 * kWarps + l]); t.amax = (float)sm[4 * kWarps + l];
        }
        warp_reduce(t, kWarps);
        acc = t;
    }
}

// ---------------------------------------------------------------- stochastic pruning (Eq. 5)
// With a = |x| and thr = fl32(alpha*eps) <= alpha, Eq. 5 is
//     out = (a >= thr) ? sign(x) * max(a, alpha) : +0
// (a > alpha passes both tests and max keeps a; thr <= a <= alpha gives alpha).
// ZCHECK adds the explicit "a zero stays zero" test that is needed only when
// alpha is so small that alpha*eps can round to zero.
template <bool ZCHECK>
__device__ __forceinline__ uint32_t prune_elem(uint32_t xb, float eps, float tau) {
    const float a = fabsf(u2f(xb));
    const float thr = __fmul_rn(tau, eps);               // one fp32 rounding, subnormals kept
    bool p = a >= thr;
    if (ZCHECK) p = p && (a != 0.f);
    const uint32_t kept = (xb & 0x80000000u) | f2u(fmaxf(a, tau));
    return p ? kept : 0u;
}

// Hot-path forms, for alpha >= kPruneFastMin.  c = alpha * 2^-16 is then exact, and
// fma(h, c, c) = fl32(c * (h + 1)) = fl32(alpha * eps): the same single rounding as
// above with one instruction less.
constexpr float kPruneFastMin = 0x1p-100f;

__device__ __forceinline__ uint32_t prune_elem_fast(uint32_t xb, float hf, float c, float tau) {
    const float a = fabsf(u2f(xb));
    const float thr = fmaf(hf, c, c);
    const uint32_t kept = (xb & 0x80000000u) | f2u(fmaxf(a, tau));
    return a >= thr ? kept : 0u;
}

// bf16, two elements of one 32-bit word at a time.  A bf16 magnitude a (pattern
// a16) and a non-negative fp32 threshold (pattern tb) compare as their patterns:
// a >= thr  <=>  (a16 << 16) >= tb  <=>  (a16 << 16) - tb >= 0 as a signed integer
// (both are below 2^31).  The two differences' sign bits, spread over their 16-bit
// lanes by one byte permute, zero the pruned lanes; max(a, alpha) is a packed
// 16-bit maximum because alpha is a bf16 value too.
__device__ __forceinline__ uint32_t prune_pair_bf16(uint32_t w, uint32_t r, float c, uint32_t tau2) {
    const float h0 = (float)(unsigned short)(r & 0xFFFFu), h1 = (float)(unsigned short)(r >> 16);
    const uint32_t mag2 = w & 0x7FFF7FFFu;
    const uint32_t d0 = (mag2 << 16) - f2u(fmaf(h0, c, c));
    const uint32_t d1 = (mag2 & 0xFFFF0000u) - f2u(fmaf(h1, c, c));
    uint32_t dead2;
    asm("prmt.b32 %0, %1, %2, 0xFFBB;" : "=r"(dead2) : "r"(d0), "r"(d1));   // sign of d0 | sign of d1, per lane
    const uint32_t kept2 = __vmaxs2(mag2, tau2) | (w & 0x80008000u);
    return kept2 & ~dead2;
}

// What an apply tile counts for its layer's result record when asked to (COUNT): pruning: a =
// outputs that are not zero, b = inputs above alpha (a - b of the kept ones were snapped to
// +-alpha); quantisation: a = codes that are not zero, b = codes of the largest magnitude.
struct TileCounts { uint32_t a = 0, b = 0; };

// Counts of one chunk of a pruning tile, taken from the input chunk and the finished output
// chunk, so that the elementwise forms above stay as they are.  Elements past the end of the
// tensor were read as zeros and written as zeros: they count in neither.
template <int DT>
__device__ __forceinline__ void count_pruned_chunk(const Chunk &in, const Chunk &o, float tau, TileCounts &tc) {
    if (DT == LGN_F32) {
        #pragma unroll
        for (int k = 0; k < 8; ++k) {
            tc.a += (o.w[k] & 0x7FFFFFFFu) != 0u ? 1u : 0u;
            tc.b += fabsf(u2f(in.w[k])) > tau ? 1u : 0u;
        }
    } else {
        const uint32_t ones = 0x00010001u, neg_tau2 = (0u - (f2u(tau) >> 16)) & 0xFFFFu;
        uint32_t a2 = 0u, b2 = 0u;                         // two 16-bit lane counters each: at most 8 per chunk
        #pragma unroll
        for (int k = 0; k < 8; ++k) {
            a2 += __vminu2(o.w[k] & 0x7FFF7FFFu, ones);
            b2 += __vminu2(__viaddmax_s16x2(in.w[k] & 0x7FFF7FFFu, neg_tau2 * ones, 0u), ones);   // max(|x| - alpha, 0) as patterns
        }
        tc.a += (a2 & 0xFFFFu) + (a2 >> 16);
        tc.b += (b2 & 0xFFFFu) + (b2 >> 16);
    }
}

// tau == 0 never reaches the fast forms' arithmetic (the tile is copied instead).
template <int DT, bool FULL, int TILE = kTileElems, bool COUNT = false>
__device__ __forceinline__ void prune_tile(const void *g, void *out, uint64_t tile_base, uint64_t n,
                                           float tau, uint64_t seed, const Weyl &wy, TileCounts *tc = nullptr) {
    constexpr int C = ElemTraits<DT>::kChunk;
    constexpr int kLoads = TILE / (kThreads * C);
    // chunks per register buffer: two for whole fp32 tiles (the pass waits for memory there, and with
    // 80 registers there is room: +0.3 % fused, +2 % alone), one otherwise
    constexpr int kGroup = (FULL && DT == LGN_F32) ? 2 : 1;
    constexpr bool ZCHECK = !FULL;                        // the general body also serves tiny thresholds
    const float c = tau * 0x1p-16f;                       // used by the hot path only (FULL: alpha >= kPruneFastMin or 0)
    const uint32_t tau2 = (f2u(tau) >> 16) * 0x00010001u; // alpha's bf16 pattern in both lanes
    pipelined_tile<DT, FULL, Ld::Stream, kLoads, kGroup>(g, tile_base, n, [&](const Chunk (&v)[kGroup], int j0) {
        #pragma unroll
        for (int j = 0; j < kGroup; ++j) {
            const uint64_t i = tile_base + (uint64_t)((j0 + j) * kThreads + threadIdx.x) * C;
            if (!FULL && i >= n) continue;
            Chunk o;
            if (tau == 0.f) {
                o = v[j];                                  // alpha = 0: the tensor is left as it is
            } else {
                uint4 rr[C / 8];
                rand_chunk<DT, FULL>(seed, i, wy, rr);
                #pragma unroll
                for (int b = 0; b < C / 8; ++b) {
                    const uint4 r = rr[b];
                    if constexpr (FULL && DT == LGN_BF16) {
                        const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
                        #pragma unroll
                        for (int pr = 0; pr < 4; ++pr) o.w[b * 4 + pr] = prune_pair_bf16(v[j].w[b * 4 + pr], rw[pr], c, tau2);
                    } else {
                        #pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const int k = b * 8 + e;
                            uint32_t res;
                            if constexpr (FULL) res = prune_elem_fast(elem_bits<DT>(v[j], k), rand_hf(r, e), c, tau);
                            else                res = prune_elem<ZCHECK>(elem_bits<DT>(v[j], k), eps_of(r, e), tau);
                            if (DT == LGN_F32) o.w[k] = res;
                            else if ((k & 1) == 0) o.w[k >> 1] = res >> 16;
                            else o.w[k >> 1] |= res & 0xFFFF0000u;
                        }
                    }
                }
            }
            store_chunk<DT, FULL>(out, i, n, o);
            if constexpr (COUNT) count_pruned_chunk<DT>(v[j], o, tau, *tc);
        }
    });
}

// ---------------------------------------------------------------- FP quantisation (Eq. 1-2, Algorithm 1)
struct QuantParams {
    int32_t  d;          // dropped fraction bits of an fp32 pattern, 23 - man_bits
    int32_t  n1;         // man_bits
    int32_t  K;          // 127 + scale_exp - E_max: fp32 exponent field minus K = code exponent field
    int32_t  nfield;     // 2^exp_bits
    uint32_t rtn_add;    // 2^(d-1) - 1
    uint32_t lsb_mask;   // 1 if man_bits > 0 else 0 (ties go to the even mantissa integer)
    uint32_t man_mask;   // 2^man_bits - 1
    uint32_t top;        // largest magnitude code
    uint32_t min_code;   // smallest normal: exponent field 1, mantissa 0
    uint32_t sign_bit;   // 1 << (nbits - 1)
    int32_t  k23;        // fast path: min(K, 255) << 23, taken off the pattern before the shift
    uint32_t sr_mult;    // fast path: 2^(d-16), places the 16 random bits below the kept bits
    float    alpha;      // smallest normal in the tensor's units, 2^(1 - E_max + scale_exp) as fp32
    uint32_t one;        // the value 1, as a run-time operand (see quant_elem)
    uint32_t pad[2];
};
static_assert(sizeof(QuantParams) == 64, "QuantParams is moved as four 16-byte words");

__host__ __device__ inline QuantParams make_quant_params(const lgn_fp_format_t &f) {
    QuantParams q;
    const int Emax = 1 << (f.exp_bits - 1);
    q.n1 = f.man_bits;
    q.d = 23 - f.man_bits;
    q.K = 127 + f.scale_exp - Emax;
    q.nfield = 1 << f.exp_bits;
    q.rtn_add = (1u << (q.d - 1)) - 1u;
    q.lsb_mask = f.man_bits > 0 ? 1u : 0u;
    q.man_mask = (1u << f.man_bits) - 1u;
    q.top = (((1u << f.exp_bits) - 1u) << f.man_bits) | q.man_mask;
    q.min_code = 1u << f.man_bits;
    q.sign_bit = 1u << (f.nbits - 1);
    q.k23 = (q.K < 0 ? 0 : (q.K > 255 ? 255 : q.K)) << 23;
    q.sr_mult = 1u << (q.d - 16);
    const int ea = 1 - Emax + f.scale_exp;               // exponent of the smallest normal
    uint32_t ab;
    if (ea > 127) ab = 0x7F800000u;                      // beyond fp32: +inf
    else if (ea >= -126) ab = (uint32_t)(ea + 127) << 23;
    else if (ea >= -149) ab = 1u << (ea + 149);          // an fp32 subnormal
    else ab = 0u;
    memcpy(&q.alpha, &ab, 4);
    q.one = 1u;
    q.pad[0] = q.pad[1] = 0u;
    return q;
}

// Code of one element from its fp32 bit pattern, integer arithmetic on the
// pattern: adding the rounding increment below the kept bits lets a mantissa
// carry run into the exponent field by itself.  h = the element's 16 random
// bits (unused for round-to-nearest).
//
// FAST (K >= 1, the usual case: the layer scale is not so small that fp32
// subnormal inputs could land inside the format's range).  With the pattern
// taken as a signed integer and K << 23 subtracted, the arithmetic shift by d
// gives [E + E_max | mantissa] directly; it is <= min_code exactly for the
// values that underflow (E <= -E_max) and > top exactly for those that clip, so
// one clamp to [min_code, top] settles both, and a value that underflows
// (|x| below the smallest normal) is then zeroed.  The additions are written as multiply-adds
// with the run-time operand q.one so that they issue on the multiply-add pipe
// and leave the integer ALU, the bottleneck of this kernel, to the shifts,
// clamps and selects.
template <bool SR, bool FAST>
__device__ __forceinline__ uint32_t quant_elem(uint32_t xb, uint32_t h, const QuantParams &q) {
    const uint32_t mag = xb & 0x7FFFFFFFu;
    const float a = u2f(mag);
    if (FAST) {
        int m2;
        if (SR) {
            const int base = (int)(mag * q.one) - q.k23;
            m2 = (int)(h * q.sr_mult) + base;
        } else {
            const uint32_t lsb = (mag >> q.d) & q.lsb_mask;
            const int base = (int)(mag * q.one) + (int)q.rtn_add - q.k23;
            m2 = (int)(lsb * q.one) + base;
        }
        const int raw = m2 >> q.d;                                        // arithmetic shift
        const uint32_t code = (uint32_t)min(max(raw, (int)q.min_code), (int)q.top);
        const bool kill = a < q.alpha;                                    // E <= -E_max: underflow
        const uint32_t comb = (xb >> 31) * q.sign_bit + code;
        return kill ? 0u : comb;
    }
    uint32_t m = mag;
    int K = q.K;
    if (m < 0x00800000u) {                               // fp32 subnormal (or zero): renormalise exactly
        m = f2u(u2f(m) * 16777216.0f);
        K += 24;
    }
    const uint32_t add = SR ? (h << (q.d - 16)) : (q.rtn_add + ((m >> q.d) & q.lsb_mask));
    const uint32_t m2 = m + add;
    const int f_pre = (int)(m >> 23) - K;                // E + E_max before rounding
    const int f_post = (int)(m2 >> 23) - K;              // ... after a possible carry
    uint32_t code = ((uint32_t)f_post << q.n1) | ((m2 >> q.d) & q.man_mask);
    if (f_post >= q.nfield) code = q.top;                // E >= E_max: clip
    if (f_pre <= 0 || mag == 0u) code = 0u;              // E <= -E_max: underflow
    return code ? (code | ((xb >> 31) ? q.sign_bit : 0u)) : 0u;
}

// bf16 fast path: two elements at a time, both halves of a 32-bit word, in
// 16-bit lanes (the element's own bf16 pattern already holds sign, the same
// 8-bit exponent field as fp32, and 7 fraction bits).  Same arithmetic as
// quant_elem's fast path with d' = 7 - man_bits dropped bits, but measured from
// the smallest normal: with lim = (K+1) << 7 (its bf16 pattern) and
// t = magnitude - lim, a lane is below the smallest normal exactly when t < 0,
// and otherwise its code is ((t + increment) >> d') + min_code, clipped to top
// (lim is a multiple of 2^d', so this equals the shifted sum minus K << man_bits).
// The packed 16-bit add-max / add-min instructions keep the lanes apart; the
// lanes with t < 0 are zeroed by a byte permute that spreads each lane's sign
// bit over the lane.  Needs 1 <= K <= 255 so that every lane value fits a signed
// 16-bit integer.
struct PackedQuant {
    uint32_t dq;        // 7 - man_bits
    uint32_t add_a;     // stochastic: lane mask of the dq random bits; nearest: 2^(dq-1) - 1 in both lanes
    uint32_t add_b;     // stochastic: 16 - dq (shift of the random word); nearest: lane mask of the kept LSB
    uint32_t keep2;     // lane mask of the 16 - dq bits left after the shift
    uint32_t min2, top2;
    uint32_t neg_lim2;  // -((K + 1) << 7) in both lanes
    uint32_t sign2;     // sign bit of a code in both lanes
};

template <bool SR>
__device__ __forceinline__ PackedQuant make_packed_quant(const QuantParams &q) {
    PackedQuant p;
    const uint32_t rep = 0x00010001u;
    p.dq = 7u - (uint32_t)q.n1;
    if (SR) { p.add_a = ((1u << p.dq) - 1u) * rep; p.add_b = 16u - p.dq; }
    else    { p.add_a = ((1u << (p.dq - 1u)) - 1u) * rep; p.add_b = q.lsb_mask * rep; }
    p.keep2 = ((1u << (16u - p.dq)) - 1u) * rep;
    p.min2 = q.min_code * rep;
    p.top2 = q.top * rep;
    p.neg_lim2 = ((0u - (((uint32_t)q.K + 1u) << 7)) & 0xFFFFu) * rep;
    p.sign2 = q.sign_bit * rep;
    return p;
}

// 0xFFFF in every 16-bit lane whose sign bit is set, 0 elsewhere.
__device__ __forceinline__ uint32_t lane_sign_mask(uint32_t x) {
    uint32_t m;
    asm("prmt.b32 %0, %1, %1, 0xBB99;" : "=r"(m) : "r"(x));   // bytes 1,1,3,3 with the sign-replicate flag
    return m;
}

template <int NBITS, bool SR>
__device__ __forceinline__ uint32_t quant_pair_bf16(uint32_t w, uint32_t r, const PackedQuant &p) {
    const uint32_t none = 0x80008000u;                            // a max() against it changes nothing
    const uint32_t mag2 = w & 0x7FFF7FFFu;
    const uint32_t t2 = __viaddmax_s16x2(mag2, p.neg_lim2, none); // magnitude - lim per lane, in [-32768, 32511]
    const uint32_t add2 = SR ? ((r >> p.add_b) & p.add_a) : (p.add_a + ((t2 >> p.dq) & p.add_b));
    const uint32_t m2 = __viaddmax_s16x2(t2, add2, none);         // per lane: no carry from a negative lane
    const uint32_t post2 = (m2 >> p.dq) & p.keep2;                // [exponent field - (K+1) | mantissa] per lane
    const uint32_t c2 = __viaddmin_s16x2(post2, p.min2, p.top2);  // min(post + min_code, top)
    const uint32_t dead2 = lane_sign_mask(t2);
    const uint32_t fin2 = (c2 | ((w >> (16 - NBITS)) & p.sign2)) & ~dead2;
    return (fin2 | (fin2 >> (16 - NBITS))) & ((1u << (2 * NBITS)) - 1u);
}

// Quantise one tile and write its slice of the packed stream.  Each lane packs
// the codes of its chunk into B = kChunk*NBITS bits (up to four 32-bit words).
// Output words are assembled from the lane in which they start and, where B is
// not a multiple of 32, the first bits of the next lane (one warp shuffle), so
// every store is an aligned 32-bit word of the little-endian bit stream.
// `total_words` = words in the whole stream.
template <int DT, int NBITS, bool SR, bool FAST, bool FULL, int TILE = kTileElems, bool COUNT = false>
__device__ __forceinline__ void quant_tile(const void *g, uint32_t *codes, uint64_t tile_base, uint64_t n,
                                           uint64_t total_words, const QuantParams &q, uint64_t seed, const Weyl &wy,
                                           TileCounts *tc = nullptr) {
    constexpr int C = ElemTraits<DT>::kChunk;
    constexpr int B = C * NBITS;                           // bits per lane per load step: 32..128
    constexpr int NW = (B + 31) / 32;                      // words that hold a lane's bits
    constexpr int kLoads = TILE / (kThreads * C);
    constexpr int kGroup = 1;
    const int lane = threadIdx.x & 31;
    const int o0 = (B % 32 == 0) ? 0 : ((32 - ((lane * B) & 31)) & 31);   // first word boundary inside this lane
    PackedQuant pq;
    if constexpr (DT == LGN_BF16 && FAST) pq = make_packed_quant<SR>(q);

    pipelined_tile<DT, FULL, Ld::Stream, kLoads, kGroup>(g, tile_base, n, [&](const Chunk (&v)[kGroup], int j0) {
        #pragma unroll
        for (int j = 0; j < kGroup; ++j) {
            const uint64_t i = tile_base + (uint64_t)((j0 + j) * kThreads + threadIdx.x) * C;
            uint32_t cw[NW + 1];
            #pragma unroll
            for (int k = 0; k <= NW; ++k) cw[k] = 0u;
            uint4 rr[C / 8];
            #pragma unroll
            for (int b = 0; b < C / 8; ++b) rr[b] = make_uint4(0u, 0u, 0u, 0u);
            if (SR) rand_chunk<DT, FULL>(seed, i, wy, rr);
            #pragma unroll
            for (int b = 0; b < C / 8; ++b) {
                const uint4 r = rr[b];
                if constexpr (DT == LGN_BF16 && FAST) {
                    const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
                    #pragma unroll
                    for (int pr = 0; pr < 4; ++pr) {       // word pr of the block <-> elements 2pr, 2pr+1
                        const uint32_t two = quant_pair_bf16<NBITS, SR>(v[j].w[b * 4 + pr], rw[pr], pq);
                        if constexpr (COUNT) {
                            const uint32_t m0 = two & (q.sign_bit - 1u), m1 = (two >> NBITS) & (q.sign_bit - 1u);
                            tc->a += (m0 != 0u ? 1u : 0u) + (m1 != 0u ? 1u : 0u);
                            tc->b += (m0 == q.top ? 1u : 0u) + (m1 == q.top ? 1u : 0u);
                        }
                        const int pos = (b * 8 + 2 * pr) * NBITS;
                        cw[pos >> 5] |= two << (pos & 31);
                        if ((pos & 31) + 2 * NBITS > 32) cw[(pos >> 5) + 1] |= two >> (32 - (pos & 31));
                    }
                } else {
                    #pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int k = b * 8 + e;
                        const uint32_t code = quant_elem<SR, FAST>(elem_bits<DT>(v[j], k), SR ? rand_h(r, e) : 0u, q);
                        if constexpr (COUNT) {
                            const uint32_t m = code & (q.sign_bit - 1u);
                            tc->a += m != 0u ? 1u : 0u;
                            tc->b += m == q.top ? 1u : 0u;
                        }
                        const int pos = k * NBITS;         // a constant once the loops are unrolled
                        cw[pos >> 5] |= code << (pos & 31);
                        if ((pos & 31) + NBITS > 32) cw[(pos >> 5) + 1] |= code >> (32 - (pos & 31));
                    }
                }
            }
            const uint64_t lane_bit = i * (uint64_t)NBITS;  // position of this lane's bit 0 in the stream
            if (B % 32 == 0) {                             // whole words per lane: no neighbour needed
                const uint64_t w0 = lane_bit >> 5;
                #pragma unroll
                for (int k = 0; k < NW; ++k)
                    if (FULL || w0 + k < total_words) st4_stream(codes + w0 + k, cw[k]);
            } else {
                // the stream seen from this lane: its own B bits, then the next lane's
                const uint32_t nx = __shfl_down_sync(0xFFFFFFFFu, cw[0], 1);
                constexpr int jB = B / 32, rB = B % 32;
                uint32_t s[NW + 1];
                #pragma unroll
                for (int k = 0; k <= NW; ++k)
                    s[k] = (k < jB) ? cw[k] : (k == jB) ? (cw[jB] | (nx << rB)) : (nx >> ((32 - rB) & 31));
                const uint64_t w0 = (lane_bit + o0) >> 5;
                #pragma unroll
                for (int k = 0; k < NW; ++k) {
                    if (o0 + 32 * k < B) {
                        const uint32_t word = __funnelshift_r(s[k], s[k + 1], o0);
                        if (FULL || w0 + k < total_words) st4_stream(codes + w0 + k, word);   // a whole tile ends on a word boundary
                    }
                }
            }
        }
    });
}

}  // namespace lgn
