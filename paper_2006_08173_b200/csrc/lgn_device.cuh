// Device-side building blocks: 16-byte tile loads, the counter-based random
// bits, and the per-tile bodies of the three O(n) passes (statistics, stochastic
// pruning, FP quantisation + packing).  One tile = kTileElems consecutive
// elements handled by one CTA of kThreads threads; in every load step thread t
// of the CTA takes the t-th 16-byte vector of a kThreads*16-byte span, so each
// warp instruction touches 512 contiguous bytes.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "lgn.h"

namespace lgn {

constexpr int kThreads   = 256;
constexpr int kWarps     = kThreads / 32;
constexpr int kTileElems = 16384;

template <int DT> struct ElemTraits;
template <> struct ElemTraits<LGN_F32>  { static constexpr int kVec = 4; static constexpr int kBytes = 4; };
template <> struct ElemTraits<LGN_BF16> { static constexpr int kVec = 8; static constexpr int kBytes = 2; };

__device__ __forceinline__ float    u2f(uint32_t u) { return __uint_as_float(u); }
__device__ __forceinline__ uint32_t f2u(float f)    { return __float_as_uint(f); }

// ---------------------------------------------------------------- loads / stores
enum class Ld { Keep, Stream };   // Keep: normal L2 policy (data is read again); Stream: evict first

template <Ld P>
__device__ __forceinline__ uint4 ld16(const void *p) {
    uint4 v;
    if (P == Ld::Keep)
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    else
        asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void st16_stream(void *p, const uint4 &v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__device__ __forceinline__ void st4_stream(void *p, uint32_t v) {
    asm volatile("st.global.cs.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

// The vector of kVec elements that starts at element index `i` (a multiple of
// kVec).  FULL: the whole vector lies inside [0, n).  Otherwise elements at or
// past n read as zero.
template <int DT, bool FULL, Ld P>
__device__ __forceinline__ uint4 load_vec(const void *g, uint64_t i, uint64_t n) {
    constexpr int V = ElemTraits<DT>::kVec;
    if (FULL || i + V <= n)
        return ld16<P>(static_cast<const char *>(g) + i * ElemTraits<DT>::kBytes);
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    if (DT == LGN_F32) {
        const uint32_t *p = static_cast<const uint32_t *>(g);
        #pragma unroll
        for (int k = 0; k < 4; ++k) if (i + k < n) w[k] = p[i + k];
    } else {
        const uint16_t *p = static_cast<const uint16_t *>(g);
        #pragma unroll
        for (int k = 0; k < 8; ++k) if (i + k < n) w[k >> 1] |= (uint32_t)p[i + k] << ((k & 1) * 16);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Store a vector of kVec output elements of the tensor's own type at element
// index i; elements at or past n are not written.
template <int DT, bool FULL>
__device__ __forceinline__ void store_vec(void *out, uint64_t i, uint64_t n, const uint4 &v) {
    constexpr int V = ElemTraits<DT>::kVec;
    if (FULL || i + V <= n) {
        st16_stream(static_cast<char *>(out) + i * ElemTraits<DT>::kBytes, v);
        return;
    }
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    if (DT == LGN_F32) {
        uint32_t *p = static_cast<uint32_t *>(out);
        #pragma unroll
        for (int k = 0; k < 4; ++k) if (i + k < n) p[i + k] = w[k];
    } else {
        uint16_t *p = static_cast<uint16_t *>(out);
        #pragma unroll
        for (int k = 0; k < 8; ++k) if (i + k < n) p[i + k] = (uint16_t)(w[k >> 1] >> ((k & 1) * 16));
    }
}

// fp32 bit pattern of element k of a vector (bf16 widened exactly).
template <int DT>
__device__ __forceinline__ uint32_t elem_bits(const uint4 &v, int k) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    if (DT == LGN_F32) return w[k];
    return (k & 1) ? (w[k >> 1] & 0xFFFF0000u) : (w[k >> 1] << 16);
}

// ---------------------------------------------------------------- random bits
// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies
// with the halves crossed and xored with the counter and a Weyl-stepped key.
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1) {
    #pragma unroll
    for (int r = 0; r < 10; ++r) {
        unsigned long long p0 = (unsigned long long)0xD2511F53u * c0;
        unsigned long long p1 = (unsigned long long)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

// The four 32-bit words of elements 4b .. 4b+3 under `seed`.
__device__ __forceinline__ uint4 rand_block(uint64_t seed, uint64_t b) {
    return philox4x32_10((uint32_t)b, (uint32_t)(b >> 32), 0u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32));
}

// ---------------------------------------------------------------- statistics
__device__ __forceinline__ float lg2_approx(float a) {
    float y;
    asm("lg2.approx.f32 %0, %1;" : "=f"(y) : "f"(a));   // subnormal inputs are handled (no .ftz)
    return y;
}

struct StatsAcc {            // per thread, in log2 units
    double s1 = 0.0, s2 = 0.0;
    unsigned long long cnt = 0;
};

// Adds one tile to the thread's accumulators.  y = log2|x| in fp32.  The sums
// are taken of d = y - P, where the pivot P is the largest y in the first run
// of this thread's elements that holds a nonzero: d stays of the order of the
// spread of the data whatever its scale, so short fp32 runs of d and d^2 lose
// nothing that matters, and a tensor whose magnitudes are all equal gives a
// variance of exactly zero.  Runs go to fp64 accumulators; the pivot is taken
// out again in fp64 at the end of the tile:
//   sum y = sum d + c P,   sum y^2 = sum d^2 + 2 P sum d + c P^2.
template <int DT, bool FULL>
__device__ __forceinline__ void stats_tile(const void *g, uint64_t tile_base, uint64_t n, StatsAcc &acc) {
    constexpr int V = ElemTraits<DT>::kVec;
    constexpr int kLoads = kTileElems / (kThreads * V);   // 16 (fp32) or 8 (bf16)
    constexpr int kGroup = 4;                             // loads in flight per thread
    constexpr int kRunVecs = 16 / V;                      // vectors per fp32 run of 16 elements
    const float kUnset = -__int_as_float(0x7F800000);     // -inf: no nonzero seen yet
    float P = kUnset;
    double D1 = 0.0, D2 = 0.0;
    unsigned long long C = 0;
    #pragma unroll 1
    for (int j0 = 0; j0 < kLoads; j0 += kGroup) {
        uint4 v[kGroup];
        #pragma unroll
        for (int j = 0; j < kGroup; ++j)
            v[j] = load_vec<DT, FULL, Ld::Keep>(g, tile_base + (uint64_t)((j0 + j) * kThreads + threadIdx.x) * V, n);
        #pragma unroll
        for (int r = 0; r < kGroup / kRunVecs; ++r) {
            float y[16];
            #pragma unroll
            for (int e = 0; e < 16; ++e)
                y[e] = lg2_approx(fabsf(u2f(elem_bits<DT>(v[r * kRunVecs + e / V], e % V))));   // -inf for zero
            if (P == kUnset) {
                #pragma unroll
                for (int e = 0; e < 16; ++e) P = fmaxf(P, y[e]);
            }
            float s1 = 0.f, s2 = 0.f;
            uint32_t c = 0;
            #pragma unroll
            for (int e = 0; e < 16; ++e) {
                bool nz = y[e] != kUnset;
                float d = nz ? y[e] - P : 0.f;
                s1 += d;
                s2 = fmaf(d, d, s2);
                c += nz ? 1u : 0u;
            }
            D1 += (double)s1;
            D2 += (double)s2;
            C += c;
        }
    }
    if (C) {
        const double p = (double)P, c = (double)C;
        acc.s1 += D1 + c * p;
        acc.s2 += D2 + p * (2.0 * D1 + c * p);
        acc.cnt += C;
    }
}

// Fixed-shape tree over the CTA; the result is valid in thread 0.
__device__ __forceinline__ void block_reduce(StatsAcc &acc, double *sm /* 3*kWarps */) {
    #pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        acc.s1 += __shfl_down_sync(0xFFFFFFFFu, acc.s1, off);
        acc.s2 += __shfl_down_sync(0xFFFFFFFFu, acc.s2, off);
        acc.cnt += __shfl_down_sync(0xFFFFFFFFu, acc.cnt, off);
    }
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    __syncthreads();                      // sm may still be in use by an earlier reduction
    if (l == 0) { sm[w] = acc.s1; sm[kWarps + w] = acc.s2; sm[2 * kWarps + w] = __longlong_as_double((long long)acc.cnt); }
    __syncthreads();
    if (w == 0) {
        StatsAcc t;
        if (l < kWarps) { t.s1 = sm[l]; t.s2 = sm[kWarps + l]; t.cnt = (unsigned long long)__double_as_longlong(sm[2 * kWarps + l]); }
        #pragma unroll
        for (int off = kWarps / 2; off > 0; off >>= 1) {
            t.s1 += __shfl_down_sync(0xFFFFFFFFu, t.s1, off);
            t.s2 += __shfl_down_sync(0xFFFFFFFFu, t.s2, off);
            t.cnt += __shfl_down_sync(0xFFFFFFFFu, t.cnt, off);
        }
        acc = t;
    }
}

// ---------------------------------------------------------------- stochastic pruning (Eq. 5)
__device__ __forceinline__ uint32_t prune_elem(uint32_t xb, uint32_t r, float tau, uint32_t tau_bits) {
    float a = fabsf(u2f(xb));
    float eps = u2f(0x3F800000u | (r >> 9)) - 1.0f;      // (r >> 9) / 2^23, exact
    float thr = __fmul_rn(tau, eps);                     // one fp32 rounding, subnormals kept
    uint32_t snapped = (xb & 0x80000000u) | tau_bits;
    bool keep = a > tau;
    bool snap = (a >= thr) && (a != 0.f);
    return keep ? xb : (snap ? snapped : 0u);
}

template <int DT, bool FULL>
__device__ __forceinline__ void prune_tile(const void *g, void *out, uint64_t tile_base, uint64_t n,
                                           float tau, uint64_t seed) {
    constexpr int V = ElemTraits<DT>::kVec;
    constexpr int kLoads = kTileElems / (kThreads * V);
    constexpr int kGroup = 4;
    const uint32_t tau_bits = f2u(tau);
    #pragma unroll 1
    for (int j0 = 0; j0 < kLoads; j0 += kGroup) {
        uint4 v[kGroup];
        #pragma unroll
        for (int j = 0; j < kGroup; ++j)
            v[j] = load_vec<DT, FULL, Ld::Stream>(g, tile_base + (uint64_t)((j0 + j) * kThreads + threadIdx.x) * V, n);
        #pragma unroll
        for (int j = 0; j < kGroup; ++j) {
            const uint64_t i = tile_base + (uint64_t)((j0 + j) * kThreads + threadIdx.x) * V;
            if (!FULL && i >= n) continue;
            uint4 o;
            if (DT == LGN_F32) {
                uint4 r = rand_block(seed, i >> 2);
                o.x = prune_elem(v[j].x, r.x, tau, tau_bits);
                o.y = prune_elem(v[j].y, r.y, tau, tau_bits);
                o.z = prune_elem(v[j].z, r.z, tau, tau_bits);
                o.w = prune_elem(v[j].w, r.w, tau, tau_bits);
            } else {
                uint4 r0 = rand_block(seed, i >> 2), r1 = rand_block(seed, (i >> 2) + 1);
                const uint32_t rr[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
                uint32_t w[4];
                #pragma unroll
                for (int k = 0; k < 4; ++k) {
                    uint32_t lo = prune_elem(elem_bits<DT>(v[j], 2 * k), rr[2 * k], tau, tau_bits);
                    uint32_t hi = prune_elem(elem_bits<DT>(v[j], 2 * k + 1), rr[2 * k + 1], tau, tau_bits);
                    w[k] = (hi & 0xFFFF0000u) | (lo >> 16);
                }
                o = make_uint4(w[0], w[1], w[2], w[3]);
            }
            store_vec<DT, FULL>(out, i, n, o);
        }
    }
}

// ---------------------------------------------------------------- FP quantisation (Eq. 1-2, Algorithm 1)
struct QuantParams {
    int32_t  d;          // dropped fraction bits, 23 - man_bits
    int32_t  n1;         // man_bits
    int32_t  K;          // 127 + scale_exp - E_max: fp32 exponent field minus K = code exponent field
    int32_t  nfield;     // 2^exp_bits
    uint32_t rtn_add;    // 2^(d-1) - 1
    uint32_t lsb_mask;   // 1 if man_bits > 0 else 0 (ties go to the even mantissa integer)
    uint32_t man_mask;   // 2^man_bits - 1
    uint32_t top;        // largest magnitude code
    uint32_t min_code;   // smallest normal: exponent field 1, mantissa 0
    uint32_t sign_bit;   // 1 << (nbits - 1)
};

__host__ __device__ inline QuantParams make_quant_params(const lgn_fp_format_t &f) {
    QuantParams q;
    q.n1 = f.man_bits;
    q.d = 23 - f.man_bits;
    q.K = 127 + f.scale_exp - (1 << (f.exp_bits - 1));
    q.nfield = 1 << f.exp_bits;
    q.rtn_add = (1u << (q.d - 1)) - 1u;
    q.lsb_mask = f.man_bits > 0 ? 1u : 0u;
    q.man_mask = (1u << f.man_bits) - 1u;
    q.top = (((1u << f.exp_bits) - 1u) << f.man_bits) | q.man_mask;
    q.min_code = 1u << f.man_bits;
    q.sign_bit = 1u << (f.nbits - 1);
    return q;
}

// Code of one element from its fp32 bit pattern; integer arithmetic on the
// pattern: adding the rounding increment below the kept bits lets a mantissa
// carry run into the exponent field by itself.
template <bool SR>
__device__ __forceinline__ uint32_t quant_elem(uint32_t xb, uint32_t r, const QuantParams &q) {
    uint32_t mag = xb & 0x7FFFFFFFu;
    uint32_t m = mag;
    int K = q.K;
    if (m < 0x00800000u) {                       // fp32 subnormal (or zero): renormalise exactly
        m = f2u(u2f(m) * 16777216.0f);
        K += 24;
    }
    uint32_t add = SR ? (r >> (32 - q.d)) : (q.rtn_add + ((m >> q.d) & q.lsb_mask));
    uint32_t m2 = m + add;
    int f_pre = (int)(m >> 23) - K;              // E + E_max before rounding
    int f_post = (int)(m2 >> 23) - K;            // ... after a possible carry
    uint32_t code = ((uint32_t)f_post << q.n1) | ((m2 >> q.d) & q.man_mask);
    if (f_post >= q.nfield) code = q.top;        // E >= E_max: clip
    if (f_pre <= 0) {                            // E <= -E_max: underflow
        if (SR) {
            int k = 1 - f_pre;                   // smallest normal is 2^k times the binade of |x'|
            uint32_t m24 = (m & 0x007FFFFFu) | 0x00800000u;
            uint32_t p = m24 >> min(k - 1, 31);
            code = ((r >> 8) < p) ? q.min_code : 0u;
        } else {
            code = 0u;
        }
    }
    if (mag == 0u) code = 0u;
    if (code != 0u) code |= (xb >> 31) ? q.sign_bit : 0u;
    return code;
}

// Quantise one tile and write its slice of the packed stream.  Each lane packs
// the codes of its own vector into B = kVec*NBITS bits; 32-bit output words are
// assembled from the lane in which they start and the one or two lanes after
// it (warp shuffles), so every store is an aligned 32-bit word of the
// little-endian bit stream.  `total_words` = words in the whole stream.
template <int DT, int NBITS, bool SR, bool FULL>
__device__ __forceinline__ void quant_tile(const void *g, uint32_t *codes, uint64_t tile_base, uint64_t n,
                                           uint64_t total_words, const QuantParams &q, uint64_t seed) {
    constexpr int V = ElemTraits<DT>::kVec;
    constexpr int B = V * NBITS;                           // bits per lane per load step
    constexpr int kLoads = kTileElems / (kThreads * V);
    constexpr int kGroup = 4;
    const int lane = threadIdx.x & 31;
    const int start = lane * B;                            // lane's first bit within the warp's span
    const int o0 = (32 - (start & 31)) & 31;               // offset of the first word that starts in this lane
    const bool has0 = o0 < B;
    const bool has1 = o0 + 32 < B;                         // only possible when B > 32 (bf16)

    #pragma unroll 1
    for (int j0 = 0; j0 < kLoads; j0 += kGroup) {
        uint4 v[kGroup];
        #pragma unroll
        for (int j = 0; j < kGroup; ++j)
            v[j] = load_vec<DT, FULL, Ld::Stream>(g, tile_base + (uint64_t)((j0 + j) * kThreads + threadIdx.x) * V, n);
        #pragma unroll
        for (int j = 0; j < kGroup; ++j) {
            const uint64_t i = tile_base + (uint64_t)((j0 + j) * kThreads + threadIdx.x) * V;
            unsigned long long c = 0;                      // this lane's B bits
            uint32_t rr[8];
            if (SR) {
                uint4 r0 = rand_block(seed, i >> 2);
                rr[0] = r0.x; rr[1] = r0.y; rr[2] = r0.z; rr[3] = r0.w;
                if (V == 8) {
                    uint4 r1 = rand_block(seed, (i >> 2) + 1);
                    rr[4] = r1.x; rr[5] = r1.y; rr[6] = r1.z; rr[7] = r1.w;
                }
            }
            #pragma unroll
            for (int k = 0; k < V; ++k) {
                uint32_t code = quant_elem<SR>(elem_bits<DT>(v[j], k), SR ? rr[k] : 0u, q);
                c |= (unsigned long long)code << (k * NBITS);
            }
            // first word of the warp's span, in units of 32-bit words of the stream
            const uint64_t lane_bit = i * (uint64_t)NBITS;  // = warp span base + start
            const uint64_t w0 = (lane_bit + o0) >> 5;
            if constexpr (B == 32) {                        // one lane, one word
                if (w0 < total_words) st4_stream(codes + w0, (uint32_t)c);
            } else if constexpr (B > 32) {
                const unsigned long long nx = __shfl_down_sync(0xFFFFFFFFu, c, 1);
                // bits [o, o+32) of (c | nx << B)
                if (has0) {
                    unsigned long long win = (c >> o0) | (B - o0 < 64 ? nx << (B - o0) : 0ull);
                    if (w0 < total_words) st4_stream(codes + w0, (uint32_t)win);
                }
                if (has1) {
                    unsigned long long win = (c >> (o0 + 32)) | (nx << (B - o0 - 32));
                    if (w0 + 1 < total_words) st4_stream(codes + w0 + 1, (uint32_t)win);
                }
            } else {
                const uint32_t c32 = (uint32_t)c;
                const uint32_t n1 = __shfl_down_sync(0xFFFFFFFFu, c32, 1);
                const uint32_t n2 = __shfl_down_sync(0xFFFFFFFFu, c32, 2);
                if (has0) {
                    unsigned long long win = (unsigned long long)c32 | ((unsigned long long)n1 << B)
                                           | ((unsigned long long)n2 << (2 * B));
                    if (w0 < total_words) st4_stream(codes + w0, (uint32_t)(win >> o0));
                }
            }
        }
    }
}

}  // namespace lgn
