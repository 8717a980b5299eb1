// Prefix code for stochastically pruned tensors (the paper's appendix
// "Encoding": 0 -> "0", +alpha -> "100", -alpha -> "101", anything else -> "11"
// followed by the FP value), fused behind Eq. 5: the encoder can apply the
// pruning itself, so the dense pruned tensor is never written.
//
// Stream format (stated in include/lgn.h): blocks of LGN_PREFIX_BLOCK elements,
// each block a run of whole 32-bit words starting at word off[b]; inside a block
// the code words of its elements follow one another in index order, stream bit k
// in bit (k mod 32) of word (k div 32), the FP value least-significant bit first.
//
// Three launches per call:
//   count  every block's length in words                      (reads the tensor)
//   scan   exclusive prefix sum of the lengths -> off[]       (one CTA)
//   emit   code words again, each thread ORs its bits into the block's image in
//          shared memory, whole words go out coalesced         (reads the tensor)
// The pruning decisions are recomputed in `emit` from the same counter-based
// random bits rather than stored in between.
#include <cmath>
#include <cstdint>
#include <cstring>

#include <cuda_runtime.h>

#include "lgn.h"
#include "lgn_closed_form.cuh"
#include "lgn_device.cuh"

namespace lgn {

constexpr int kPfxThreads = 256;
constexpr int kPfxPerThread = 8;                               // one block of random bits per thread
static_assert(kPfxThreads * kPfxPerThread == (int)LGN_PREFIX_BLOCK, "a CTA pass covers one block");
constexpr int kPfxWarps = kPfxThreads / 32;

template <int DT> struct PfxTraits;
template <> struct PfxTraits<LGN_F32>  { static constexpr int kWidth = 32; static constexpr uint32_t kSign = 0x80000000u; };
template <> struct PfxTraits<LGN_BF16> { static constexpr int kWidth = 16; static constexpr uint32_t kSign = 0x8000u; };

// alpha as the kernels use it: host value, or the tau field of a layer result on the device
__device__ __forceinline__ float pfx_tau(float tau_host, const lgn_layer_result_t *from) {
    return from ? (float)*(const volatile double *)&from->tau : tau_host;
}

// Storage patterns of the 8 elements that start at element index i (a multiple of 8); past n: +0.
template <int DT>
__device__ __forceinline__ void pfx_load(const void *g, uint64_t i, uint64_t n, uint32_t (&p)[kPfxPerThread]) {
    if (i + kPfxPerThread <= n) {
        if (DT == LGN_F32) {
            const uint4 a = __ldg(reinterpret_cast<const uint4 *>(static_cast<const uint32_t *>(g) + i));
            const uint4 b = __ldg(reinterpret_cast<const uint4 *>(static_cast<const uint32_t *>(g) + i) + 1);
            p[0] = a.x; p[1] = a.y; p[2] = a.z; p[3] = a.w; p[4] = b.x; p[5] = b.y; p[6] = b.z; p[7] = b.w;
        } else {
            const uint4 a = __ldg(reinterpret_cast<const uint4 *>(static_cast<const uint16_t *>(g) + i));
            const uint32_t w[4] = {a.x, a.y, a.z, a.w};
            #pragma unroll
            for (int k = 0; k < 8; ++k) p[k] = (w[k >> 1] >> ((k & 1) * 16)) & 0xFFFFu;
        }
    } else {
        #pragma unroll
        for (int k = 0; k < 8; ++k) {
            p[k] = 0u;
            if (i + k < n) p[k] = DT == LGN_F32 ? static_cast<const uint32_t *>(g)[i + k]
                                                : (uint32_t)static_cast<const uint16_t *>(g)[i + k];
        }
    }
}

// Eq. 5 on storage patterns (PRUNE), or the patterns as they are.
template <int DT, bool PRUNE>
__device__ __forceinline__ void pfx_values(uint32_t (&p)[kPfxPerThread], uint64_t i, float tau, uint64_t seed,
                                           const Weyl &wy) {
    if (!PRUNE || tau == 0.f) return;
    const uint4 r = rand_block(seed, i >> 3, wy);
    if (tau >= kPruneFastMin) {                                   // same values, cheaper form (see prune_elem_fast)
        const float c = tau * 0x1p-16f;
        #pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t xb = DT == LGN_F32 ? p[k] : p[k] << 16;
            const uint32_t res = prune_elem_fast(xb, rand_hf(r, k), c, tau);
            p[k] = DT == LGN_F32 ? res : res >> 16;
        }
    } else {
        #pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t xb = DT == LGN_F32 ? p[k] : p[k] << 16;
            const uint32_t res = prune_elem<true>(xb, eps_of(r, k), tau);
            p[k] = DT == LGN_F32 ? res : res >> 16;
        }
    }
}

// Code word of one stored pattern: its bits (first stream bit in bit 0) and its
// length.  An FP value is returned as the two prefix bits; the caller appends
// the pattern.
template <int DT>
__device__ __forceinline__ uint32_t pfx_len(uint32_t pat, uint32_t tau_pat) {
    if (pat == 0u) return 1u;
    if (tau_pat != 0u && (pat & ~PfxTraits<DT>::kSign) == tau_pat) return 3u;
    return 2u + PfxTraits<DT>::kWidth;
}

template <int DT>
__device__ __forceinline__ uint32_t tau_pattern(float tau) {
    return DT == LGN_F32 ? f2u(tau) : f2u(tau) >> 16;
}

template <int DT, bool PRUNE>
__global__ void __launch_bounds__(kPfxThreads)
prefix_count_kernel(const void *g, uint64_t n, uint64_t nblocks, float tau_host, const lgn_layer_result_t *tau_from,
                    uint64_t seed, Weyl wy, uint32_t *block_words) {
    __shared__ uint32_t sm_total[2];
    const float tau = pfx_tau(tau_host, tau_from);
    const uint32_t tp = tau_pattern<DT>(tau);
    if (threadIdx.x < 2) sm_total[threadIdx.x] = 0u;
    __syncthreads();
    uint32_t p[kPfxPerThread], q[kPfxPerThread];
    uint64_t b = blockIdx.x;
    if (b < nblocks) pfx_load<DT>(g, b * LGN_PREFIX_BLOCK + (uint64_t)threadIdx.x * kPfxPerThread, n, p);
    for (uint32_t it = 0; b < nblocks; b += gridDim.x, ++it) {
        const uint64_t i = b * LGN_PREFIX_BLOCK + (uint64_t)threadIdx.x * kPfxPerThread;
        const uint64_t bn = b + gridDim.x;                       // the next block's loads fly while this one is counted
        if (bn < nblocks) pfx_load<DT>(g, bn * LGN_PREFIX_BLOCK + (uint64_t)threadIdx.x * kPfxPerThread, n, q);
        pfx_values<DT, PRUNE>(p, i, tau, seed, wy);
        uint32_t bits = 0u;
        if ((b + 1) * LGN_PREFIX_BLOCK <= n) {                   // the whole block lies inside the tensor
            #pragma unroll
            for (int k = 0; k < 8; ++k) bits += pfx_len<DT>(p[k], tp);
        } else {
            #pragma unroll
            for (int k = 0; k < 8; ++k) if (i + k < n) bits += pfx_len<DT>(p[k], tp);
        }
        bits = __reduce_add_sync(0xFFFFFFFFu, bits);
        if ((threadIdx.x & 31) == 0) atomicAdd(&sm_total[it & 1], bits);
        __syncthreads();
        if (threadIdx.x == 0) {
            block_words[b] = (sm_total[it & 1] + 31u) >> 5;
            sm_total[it & 1] = 0u;                               // used again two blocks on, after the next barrier
        }
        #pragma unroll
        for (int k = 0; k < 8; ++k) p[k] = q[k];
    }
}

// Exclusive prefix sum of block_words[0..nblocks) into off[0..nblocks]; one CTA.
// Thread t owns the entries [t*per, (t+1)*per), per a multiple of 4 (16-byte loads).
constexpr int kScanThreads = 1024;
__global__ void __launch_bounds__(kScanThreads)
prefix_scan_kernel(const uint32_t *block_words, uint64_t nblocks, uint64_t *off) {
    __shared__ unsigned long long sm[kScanThreads / 32];
    const uint64_t per = ((nblocks + kScanThreads - 1) / kScanThreads + 3) / 4 * 4;
    const uint64_t lo = (uint64_t)threadIdx.x * per < nblocks ? (uint64_t)threadIdx.x * per : nblocks;
    const uint64_t hi = lo + per < nblocks ? lo + per : nblocks;
    unsigned long long s = 0;
    uint64_t k = lo;
    for (; k + 4 <= hi; k += 4) {                                // lo is a multiple of 4: aligned
        const uint4 v = *reinterpret_cast<const uint4 *>(block_words + k);
        s += (unsigned long long)v.x + v.y + v.z + v.w;
    }
    for (; k < hi; ++k) s += block_words[k];
    // inclusive scan of s over the CTA: warp shuffles, then the 32 warp totals
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long incl = s;
    #pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned long long v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += v;
    }
    if (lane == 31) sm[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        unsigned long long w = sm[lane];
        #pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long v = __shfl_up_sync(0xFFFFFFFFu, w, d);
            if (lane >= d) w += v;
        }
        sm[lane] = w;                                            // inclusive over warps
    }
    __syncthreads();
    unsigned long long run = incl - s + (warp ? sm[warp - 1] : 0ull);
    for (k = lo; k + 4 <= hi; k += 4) {
        const uint4 v = *reinterpret_cast<const uint4 *>(block_words + k);
        off[k] = run; off[k + 1] = run + v.x; off[k + 2] = run + v.x + v.y; off[k + 3] = run + v.x + v.y + v.z;
        run += (unsigned long long)v.x + v.y + v.z + v.w;
    }
    for (; k < hi; ++k) { off[k] = run; run += block_words[k]; }
    if (threadIdx.x == kScanThreads - 1) off[nblocks] = sm[kScanThreads / 32 - 1];
}

constexpr int kPfxImageWords = (LGN_PREFIX_BLOCK * 34u + 31u) / 32u + 2u;   // a block of FP values, plus slack

// A thread's code words, assembled in a 64-bit register that starts at the
// thread's bit position inside its first image word; every completed 32-bit word
// is ORed into the image (the first and last word of a thread are shared with its
// neighbours; words that are all zero -- runs of "0" codes -- need no write).
// nvalid = how many of the 8 elements exist (8 except in the tensor's last block).
template <int DT>
__device__ __forceinline__ void pfx_emit_thread(const uint32_t (&p)[kPfxPerThread], uint32_t tp, uint32_t pos,
                                                uint32_t nvalid, uint32_t *img) {
    constexpr uint32_t kSign = PfxTraits<DT>::kSign;
    // Two 32-bit registers hold the bits from the current image word on; `tot` is
    // the thread's bit position in the image.  Written without branches (selects
    // and a predicated shared-memory OR): the lanes of a warp would take different
    // paths at almost every element otherwise.
    const uint32_t img_addr = (uint32_t)__cvta_generic_to_shared(img);
    uint32_t lo = 0u, hi = 0u, tot = pos;
    auto append = [&](uint32_t x, uint32_t len) {                // x has `len` bits; the low register has room
        const uint32_t s = tot & 31u;
        lo |= x << s;
        hi |= __funnelshift_l(x, 0u, s);                         // x >> (32 - s), and 0 for s = 0
        const uint32_t after = tot + len;
        const uint32_t full = (after ^ tot) & 32u;               // the low register's word is complete
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\tsetp.ne.and.u32 p, %1, 0, p;\n\t"
                     "@p red.shared.or.b32 [%0], %1;\n\t}"
                     :: "r"(img_addr + (tot >> 5) * 4u), "r"(lo), "r"(full) : "memory");
        lo = full ? hi : lo;
        hi = full ? 0u : hi;
        tot = after;
    };
    #pragma unroll
    for (int k = 0; k < 8; ++k) {
        const bool in = (uint32_t)k < nvalid;
        const uint32_t pat = p[k];
        const bool zero = pat == 0u;
        const bool alpha = tp != 0u && (pat & ~kSign) == tp;
        const bool value = in && !zero && !alpha;
        const uint32_t v = zero ? 0u : alpha ? ((pat & kSign) ? 5u : 1u) : 3u;       // first stream bit in bit 0
        append(in ? v : 0u, !in ? 0u : zero ? 1u : alpha ? 3u : 2u);
        append(value ? pat : 0u, value ? (uint32_t)PfxTraits<DT>::kWidth : 0u);
    }
    if (lo) atomicOr(&img[tot >> 5], lo);
}

template <int DT, bool PRUNE>
__global__ void __launch_bounds__(kPfxThreads)
prefix_emit_kernel(const void *g, uint64_t n, uint64_t nblocks, float tau_host, const lgn_layer_result_t *tau_from,
                   uint64_t seed, Weyl wy, const uint64_t *off, uint32_t *stream, uint64_t capacity_words) {
    __shared__ uint32_t img[kPfxImageWords];
    __shared__ uint32_t sm[kPfxWarps];
    const float tau = pfx_tau(tau_host, tau_from);
    const uint32_t tp = tau_pattern<DT>(tau);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t p[kPfxPerThread], q[kPfxPerThread];
    if (blockIdx.x < nblocks)
        pfx_load<DT>(g, (uint64_t)blockIdx.x * LGN_PREFIX_BLOCK + (uint64_t)threadIdx.x * kPfxPerThread, n, p);
    for (uint64_t b = blockIdx.x; b < nblocks; b += gridDim.x) {
        const uint64_t w0 = off[b], w1 = off[b + 1];
        const uint32_t words = (uint32_t)(w1 - w0);
        const uint64_t i = b * LGN_PREFIX_BLOCK + (uint64_t)threadIdx.x * kPfxPerThread;
        const uint64_t bn = b + gridDim.x;                       // the next block's loads fly while this one is packed
        if (bn < nblocks) pfx_load<DT>(g, bn * LGN_PREFIX_BLOCK + (uint64_t)threadIdx.x * kPfxPerThread, n, q);
        if (w1 > capacity_words) {                               // does not fit: the caller sees off[nblocks] > capacity
            #pragma unroll
            for (int k = 0; k < 8; ++k) p[k] = q[k];
            continue;
        }
        for (uint32_t k = threadIdx.x; k < words + 1u; k += kPfxThreads) img[k] = 0u;
        pfx_values<DT, PRUNE>(p, i, tau, seed, wy);
        const bool full = (b + 1) * LGN_PREFIX_BLOCK <= n;
        const uint32_t nvalid = full ? 8u : (i >= n ? 0u : (n - i < 8u ? (uint32_t)(n - i) : 8u));
        uint32_t bits = 0u;
        #pragma unroll
        for (int k = 0; k < 8; ++k) if ((uint32_t)k < nvalid) bits += pfx_len<DT>(p[k], tp);
        // exclusive scan of `bits` over the CTA: warp scan, then the warp totals
        uint32_t incl = bits;
        #pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += v;
        }
        if (lane == 31) sm[warp] = incl;
        __syncthreads();                                         // also: the image is zeroed
        uint32_t pos = incl - bits;
        #pragma unroll
        for (int w = 0; w < kPfxWarps; ++w) if (w < warp) pos += sm[w];
        if (full) pfx_emit_thread<DT>(p, tp, pos, 8u, img);
        else      pfx_emit_thread<DT>(p, tp, pos, nvalid, img);
        __syncthreads();
        for (uint32_t k = threadIdx.x; k < words; k += kPfxThreads) stream[w0 + k] = img[k];
        __syncthreads();                                         // the image and sm are reused by the next block
        #pragma unroll
        for (int k = 0; k < 8; ++k) p[k] = q[k];
    }
}

// One thread decodes one block.
template <int DT>
__global__ void __launch_bounds__(128)
prefix_decode_kernel(const uint32_t *stream, const uint64_t *off, uint64_t n, uint64_t nblocks, float tau_host,
                     const lgn_layer_result_t *tau_from, void *out) {
    const uint64_t b = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= nblocks) return;
    const uint32_t tp = tau_pattern<DT>(pfx_tau(tau_host, tau_from));
    const uint32_t *p = stream + off[b], *end = stream + off[b + 1];
    unsigned long long buf = 0ull;
    int have = 0;
    const uint64_t i0 = b * LGN_PREFIX_BLOCK;
    const uint64_t i1 = i0 + LGN_PREFIX_BLOCK < n ? i0 + LGN_PREFIX_BLOCK : n;
    auto refill = [&]() {                                        // keeps 33..64 bits in hand (zeros past the block)
        if (have <= 32) {
            const unsigned long long w = p < end ? *p : 0u;
            ++p;
            buf |= w << have;
            have += 32;
        }
    };
    for (uint64_t i = i0; i < i1; ++i) {
        refill();
        uint32_t pat;
        if ((buf & 1ull) == 0ull)      { pat = 0u; buf >>= 1; have -= 1; }
        else if ((buf & 2ull) == 0ull) { pat = (buf & 4ull) ? (tp | PfxTraits<DT>::kSign) : tp; buf >>= 3; have -= 3; }
        else {
            buf >>= 2; have -= 2;
            refill();                                            // now at least 32 bits: the whole value
            pat = (uint32_t)buf & (DT == LGN_F32 ? 0xFFFFFFFFu : 0xFFFFu);
            buf >>= PfxTraits<DT>::kWidth; have -= PfxTraits<DT>::kWidth;
        }
        if (DT == LGN_F32) static_cast<uint32_t *>(out)[i] = pat;
        else               static_cast<uint16_t *>(out)[i] = (uint16_t)pat;
    }
}

static bool aligned_to(const void *p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Resident CTAs of a grid-stride kernel: SM count x CTAs per SM, at most one CTA per block of work.
template <class K>
static unsigned resident_grid(K kernel, uint64_t nblocks) {
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kPfxThreads, 0) != cudaSuccess) return 0;
    if (per_sm < 1) per_sm = 1;
    const uint64_t g = (uint64_t)sms * (uint64_t)per_sm;
    return (unsigned)(nblocks < g ? nblocks : g);
}

}  // namespace lgn

using namespace lgn;

extern "C" uint64_t lgn_prefix_blocks(uint64_t n) { return (n + LGN_PREFIX_BLOCK - 1) / LGN_PREFIX_BLOCK; }

extern "C" uint64_t lgn_prefix_bound_words(uint64_t n, lgn_dtype dt) {
    const uint64_t per = (dt == LGN_BF16 ? 16u : 32u) + 2u;
    const uint64_t full = n / LGN_PREFIX_BLOCK, rest = n % LGN_PREFIX_BLOCK;
    return full * ((LGN_PREFIX_BLOCK * per + 31) / 32) + (rest * per + 31) / 32;
}

extern "C" size_t lgn_prefix_workspace_bytes(uint64_t n) {
    return (size_t)((lgn_prefix_blocks(n) * 4 + 255) / 256 * 256 + 256);
}

extern "C" lgn_status lgn_prefix_encode(const void *g, uint64_t n, lgn_dtype dt, double tau, uint64_t seed,
                                        int apply_prune, const lgn_layer_result_t *tau_from_dev,
                                        uint32_t *stream_dev, uint64_t capacity_words, uint64_t *off_dev,
                                        void *ws, size_t ws_bytes, void *stream) {
    if (dt != LGN_F32 && dt != LGN_BF16) return LGN_ERR_INVALID_ARG;
    if (n > 0 && (g == nullptr || !aligned_to(g, 32))) return LGN_ERR_INVALID_ARG;
    if (off_dev == nullptr || !aligned_to(off_dev, 8)) return LGN_ERR_INVALID_ARG;
    if (capacity_words > 0 && (stream_dev == nullptr || !aligned_to(stream_dev, 4))) return LGN_ERR_INVALID_ARG;
    if (!(tau >= 0.0) || !std::isfinite(tau)) return LGN_ERR_INVALID_ARG;
    if (n > (1ull << 34)) return LGN_ERR_UNSUPPORTED;
    if (ws == nullptr || !aligned_to(ws, 16) || ws_bytes < lgn_prefix_workspace_bytes(n)) return LGN_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint64_t nb = lgn_prefix_blocks(n);
    uint32_t *bw = static_cast<uint32_t *>(ws);
    const float tau_used = dt == LGN_BF16 ? snap_threshold_bf16(tau) : snap_threshold_f32(tau);
    const Weyl wy = { kWeyl0, kWeyl1 };
    if (nb > 0) {
        #define LGN_PFX1(K, D, P, ...) { const unsigned grid = resident_grid(K<D, P>, nb); \
                                         if (grid == 0) return LGN_ERR_CUDA; \
                                         K<D, P><<<grid, kPfxThreads, 0, st>>>(__VA_ARGS__); }
        #define LGN_PFX(K, ...) \
            if (dt == LGN_F32) { if (apply_prune) LGN_PFX1(K, LGN_F32, true, __VA_ARGS__) else LGN_PFX1(K, LGN_F32, false, __VA_ARGS__) } \
            else               { if (apply_prune) LGN_PFX1(K, LGN_BF16, true, __VA_ARGS__) else LGN_PFX1(K, LGN_BF16, false, __VA_ARGS__) }
        LGN_PFX(prefix_count_kernel, g, n, nb, tau_used, tau_from_dev, seed, wy, bw)
        prefix_scan_kernel<<<1, kScanThreads, 0, st>>>(bw, nb, off_dev);
        LGN_PFX(prefix_emit_kernel, g, n, nb, tau_used, tau_from_dev, seed, wy, off_dev, stream_dev, capacity_words)
        #undef LGN_PFX
        #undef LGN_PFX1
    } else {
        prefix_scan_kernel<<<1, kScanThreads, 0, st>>>(bw, 0, off_dev);
    }
    return cudaGetLastError() == cudaSuccess ? LGN_OK : LGN_ERR_CUDA;
}

extern "C" lgn_status lgn_prefix_decode(const uint32_t *stream_dev, const uint64_t *off_dev, uint64_t n, lgn_dtype dt,
                                        double tau, const lgn_layer_result_t *tau_from_dev, void *out_dev,
                                        void *stream) {
    if (dt != LGN_F32 && dt != LGN_BF16) return LGN_ERR_INVALID_ARG;
    if (off_dev == nullptr || !aligned_to(off_dev, 8)) return LGN_ERR_INVALID_ARG;
    if (n > 0 && (out_dev == nullptr || stream_dev == nullptr || !aligned_to(stream_dev, 4) || !aligned_to(out_dev, 4)))
        return LGN_ERR_INVALID_ARG;
    if (!(tau >= 0.0) || !std::isfinite(tau)) return LGN_ERR_INVALID_ARG;
    if (n > (1ull << 34)) return LGN_ERR_UNSUPPORTED;
    if (n == 0) return LGN_OK;
    const uint64_t nb = lgn_prefix_blocks(n);
    const float tau_used = dt == LGN_BF16 ? snap_threshold_bf16(tau) : snap_threshold_f32(tau);
    const unsigned grid = (unsigned)((nb + 127) / 128);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dt == LGN_F32) prefix_decode_kernel<LGN_F32><<<grid, 128, 0, st>>>(stream_dev, off_dev, n, nb, tau_used, tau_from_dev, out_dev);
    else               prefix_decode_kernel<LGN_BF16><<<grid, 128, 0, st>>>(stream_dev, off_dev, n, nb, tau_used, tau_from_dev, out_dev);
    return cudaGetLastError() == cudaSuccess ? LGN_OK : LGN_ERR_CUDA;
}
