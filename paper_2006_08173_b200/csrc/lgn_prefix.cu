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
// One pass over the tensor (a memset of the small workspace, then one launch): each
// CTA encodes whole blocks into an image in shared memory, obtains the block's
// first word by a decoupled look-back over the lengths the preceding blocks have
// published, and writes the image out with coalesced stores.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <type_traits>

#include <cuda_runtime.h>

#include "lgn.h"
#include "lgn_closed_form.cuh"
#include "lgn_device.cuh"
#include "lgn_log.h"

namespace lgn {

constexpr int kPfxThreads = 256;
constexpr int kPfxPerThread = 8;                               // one block of random bits per thread
static_assert(kPfxThreads * kPfxPerThread == (int)LGN_PREFIX_BLOCK, "a CTA pass covers one block");
constexpr int kPfxWarps = kPfxThreads / 32;
constexpr int kPfxImageWords = (LGN_PREFIX_BLOCK * 34u + 31u) / 32u + 4u;   // a block of FP values, plus slack

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

template <int DT>
__device__ __forceinline__ uint32_t tau_pattern(float tau) {
    return DT == LGN_F32 ? f2u(tau) : f2u(tau) >> 16;
}

// ------------------------------------------------------------------ single-pass encoder
// Blocks are handed out in index order by a ticket counter, so every block a CTA
// may have to wait for is already in the hands of a running CTA.  Per block:
//   1. load, prune (Eq. 5), classify; every thread assembles the short codes of its
//      eight elements ("0", "100"/"101", or the "11" in front of a value: at most 24
//      bits) in one register and notes where the values cut that string;
//   2. a scan of the threads' bit counts over the CTA gives each thread's position
//      and the block's length in words, which is published as this block's
//      AGGREGATE;
//   3. the threads OR their bits into the block's image in shared memory: for each
//      value one 64-bit piece (the short bits since the previous value, then the
//      value), then the remaining short bits;
//   4. meanwhile warp 0 looks back over the preceding blocks' published lengths
//      (decoupled look-back: an INCLUSIVE prefix ends the walk) to get the block's
//      first word, publishes its own inclusive prefix, and the image goes out with
//      coalesced stores.
// Waits in the look-back are bounded; if one runs out every CTA stops and
// off[nblocks] is set to all ones.
struct PfxCtl { uint32_t ticket, error, pad[62]; };
static_assert(sizeof(PfxCtl) == 256, "control block");
constexpr unsigned long long kPfxAggregate = 1ull, kPfxInclusive = 2ull;
constexpr uint32_t kPfxMaxPolls = 1u << 20;

// A block's state word carries everything a successor needs (flag and length in one
// aligned 64-bit word) and nothing else is read through it, so relaxed accesses at
// gpu scope are enough.
__device__ __forceinline__ unsigned long long ld_state(const unsigned long long *p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_state(unsigned long long *p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}

// OR a word into the image unless it is zero: a compare and a predicated shared-memory
// reduction, no branch (most words of most lanes are zero).
__device__ __forceinline__ void pfx_or_word(uint32_t addr, uint32_t v) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %1, 0;\n\t@p red.shared.or.b32 [%0], %1;\n\t}"
                 :: "r"(addr), "r"(v) : "memory");
}

// OR the bits of x (bits above its length are zero) into the image at bit position `at`.
__device__ __forceinline__ void pfx_or64(uint32_t img_addr, uint32_t at, unsigned long long x) {
    const uint32_t s = at & 31u, a = img_addr + (at >> 5) * 4u;
    const uint32_t lo = (uint32_t)x, hi = (uint32_t)(x >> 32);
    pfx_or_word(a, lo << s);
    pfx_or_word(a + 4u, __funnelshift_l(lo, hi, s));
    pfx_or_word(a + 8u, __funnelshift_l(hi, 0u, s));
}
__device__ __forceinline__ void pfx_or32(uint32_t img_addr, uint32_t at, uint32_t x) {
    const uint32_t s = at & 31u, a = img_addr + (at >> 5) * 4u;
    pfx_or_word(a, x << s);
    pfx_or_word(a + 4u, __funnelshift_l(x, 0u, s));
}

template <int DT, bool PRUNE>
__global__ void __launch_bounds__(kPfxThreads)
prefix_encode_kernel(const void *g, uint64_t n, uint64_t nblocks, float tau_host, const lgn_layer_result_t *tau_from,
                     uint64_t seed, Weyl wy, PfxCtl *ctl, unsigned long long *state, uint64_t *off, uint32_t *stream,
                     uint64_t capacity_words) {
    constexpr uint32_t kSign = PfxTraits<DT>::kSign;
    constexpr uint32_t W = PfxTraits<DT>::kWidth;
    __shared__ uint32_t img[kPfxImageWords];
    __shared__ uint32_t pay[kPfxPerThread][kPfxThreads];         // the threads' (pruned) patterns, one column each
    __shared__ uint32_t sm_scan[kPfxWarps];
    __shared__ unsigned long long sm_ticket, sm_excl;
    const float tau = pfx_tau(tau_host, tau_from);
    const uint32_t tp = tau_pattern<DT>(tau);
    const uint32_t tpc = tp ? tp : kSign;                        // a pattern no magnitude equals: no alpha codes when alpha = 0
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    for (;;) {
        if (threadIdx.x == 0) sm_ticket = atomicAdd(&ctl->ticket, 1u);
        __syncthreads();                                         // also: the previous block's image has gone out
        const uint64_t b = sm_ticket;
        if (b >= nblocks) break;
        const uint64_t i = b * LGN_PREFIX_BLOCK + (uint64_t)threadIdx.x * kPfxPerThread;
        uint32_t p[kPfxPerThread];
        pfx_load<DT>(g, i, n, p);
        pfx_values<DT, PRUNE>(p, i, tau, seed, wy);
        const uint32_t nvalid = i >= n ? 0u : (n - i < 8u ? (uint32_t)(n - i) : 8u);

        // short codes of the eight elements, first stream bit in bit 0
        uint32_t sb = 0u, q = 0u, vm = 0u;
        unsigned long long cuts = 0ull;                          // 5 bits per element: q after the element
        auto classify = [&](auto whole) {                        // whole: all eight elements exist (every block but the last)
            #pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t pat = p[k];
                const bool in = decltype(whole)::value || (uint32_t)k < nvalid;
                const bool nz = in && pat != 0u;
                const bool al = in && (pat & ~kSign) == tpc;
                const uint32_t code = al ? ((pat & kSign) ? 5u : 1u) : (nz ? 3u : 0u);
                sb |= code << q;
                q += (in ? 1u : 0u) + (nz ? 1u : 0u) + (al ? 1u : 0u);
                if (nz && !al) vm |= 1u << k;
                cuts |= (unsigned long long)q << (5 * k);
                pay[k][threadIdx.x] = pat;
            }
        };
        if ((b + 1) * LGN_PREFIX_BLOCK <= n) classify(std::true_type{});
        else classify(std::false_type{});
        const uint32_t bits = q + W * __popc(vm);

        // exclusive scan of `bits` over the CTA
        uint32_t incl = bits;
        #pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += v;
        }
        if (lane == 31) sm_scan[warp] = incl;
        __syncthreads();
        uint32_t pos = incl - bits, total = 0u;
        #pragma unroll
        for (int w = 0; w < kPfxWarps; ++w) { const uint32_t t = sm_scan[w]; if (w < warp) pos += t; total += t; }
        const uint32_t words = (total + 31u) >> 5;
        if (threadIdx.x == 0) {
            if (b == 0) { st_state(state, ((unsigned long long)words << 2) | kPfxInclusive); sm_excl = 0ull; }
            else        st_state(state + b, ((unsigned long long)words << 2) | kPfxAggregate);
        }
        for (uint32_t k = threadIdx.x; k < words + 2u; k += kPfxThreads) img[k] = 0u;
        __syncthreads();

        // the thread's bits into the image
        const uint32_t img_addr = (uint32_t)__cvta_generic_to_shared(img);
        // One trip per value of the thread (a warp makes as many trips as its busiest lane
        // has values, about three at 8 % values, instead of eight trips over the elements);
        // the value is fetched from the thread's own column of `pay` by its index.
        uint32_t cur = pos, done = 0u;
        for (uint32_t m = vm; m; m &= m - 1u) {
            const int k = __ffs(m) - 1;
            const uint32_t cut = (uint32_t)(cuts >> (5 * k)) & 31u;
            const uint32_t plen = cut - done;                    // 2..26: ends with the value's "11"
            const uint32_t piece = (sb >> done) & ((1u << plen) - 1u);
            const uint32_t val = pay[k][threadIdx.x];
            pfx_or64(img_addr, cur, (unsigned long long)piece | ((unsigned long long)val << plen));
            cur += plen + W;
            done = cut;
        }
        if (q > done) pfx_or32(img_addr, cur, sb >> done);

        // warp 0: first word of this block = sum of the lengths of all earlier blocks
        if (warp == 0 && b > 0) {
            unsigned long long excl = 0ull;
            bool fail = false;
            for (long long j = (long long)b - 1;; j -= 32) {
                const long long idx = j - lane;
                unsigned long long v = kPfxInclusive;            // before block 0: an inclusive prefix of 0
                uint32_t polls = 0;
                for (;;) {
                    if (idx >= 0) v = ld_state(state + idx);
                    if (!__any_sync(0xFFFFFFFFu, (v & 3ull) == 0ull)) break;
                    const bool stop = ++polls > kPfxMaxPolls || *(volatile uint32_t *)&ctl->error != 0u;
                    if (__any_sync(0xFFFFFFFFu, stop)) { fail = true; break; }
                    __nanosleep(64);
                }
                if (fail) break;
                const uint32_t inc_mask = __ballot_sync(0xFFFFFFFFu, (v & 3ull) == kPfxInclusive);
                const int first = inc_mask ? __ffs(inc_mask) - 1 : 32;       // nearest block with an inclusive prefix
                unsigned long long c = lane <= first ? (v >> 2) : 0ull;
                #pragma unroll
                for (int d = 16; d > 0; d >>= 1) c += __shfl_down_sync(0xFFFFFFFFu, c, d);
                excl += __shfl_sync(0xFFFFFFFFu, c, 0);
                if (inc_mask) break;
            }
            if (lane == 0) {
                if (fail) { atomicExch(&ctl->error, 1u); sm_excl = ~0ull; }
                else      { st_state(state + b, ((excl + words) << 2) | kPfxInclusive); sm_excl = excl; }
            }
        }
        __syncthreads();                                         // the image is complete, the offset known
        const unsigned long long w0 = sm_excl;
        if (w0 == ~0ull) {                                       // a wait ran out: tell the caller and stop
            if (threadIdx.x == 0) off[nblocks] = ~0ull;
            break;
        }
        if (threadIdx.x == 0) {
            off[b] = w0;
            if (b + 1 == nblocks) off[nblocks] = w0 + words;
        }
        if (w0 + words <= capacity_words)                        // else: the caller sees off[nblocks] > capacity
            for (uint32_t k = threadIdx.x; k < words; k += kPfxThreads) stream[w0 + k] = img[k];
    }
}

__global__ void prefix_empty_kernel(uint64_t *off) { off[0] = 0ull; }

// One thread decodes one block (the code is sequential within a block); a warp takes 32
// consecutive blocks and moves in rounds of 32 elements per block.  Per round:
//   1. the warp copies, row by row with coalesced loads, the next 40 words of each of its 32
//      streams into shared memory (32 elements take at most 32 x 34 bits = 34 words, plus
//      the two words a 64-bit window may reach past its first);
//   2. every lane decodes 32 elements of its block from its row, without a branch: a 64-bit
//      window at the current bit, the class from its two low bits, the value from the bits
//      behind them, the length added to the bit position;
//   3. the warp writes the 32 rows of decoded elements out, one coalesced store per row.
// The re-read of words a slow stream has not consumed yet hits L1; no load sits on the
// decode chain.
constexpr int kDecThreads = 128;
constexpr int kDecRowWords = 40;
template <int DT>
__global__ void __launch_bounds__(kDecThreads)
prefix_decode_kernel(const uint32_t *stream, const uint64_t *off, uint64_t n, uint64_t nblocks, float tau_host,
                     const lgn_layer_result_t *tau_from, void *out) {
    constexpr uint32_t W = PfxTraits<DT>::kWidth;
    __shared__ uint32_t tile[kDecThreads / 32][32][33];
    __shared__ uint32_t rows[kDecThreads / 32][32][kDecRowWords + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint64_t b0 = ((uint64_t)blockIdx.x * kDecThreads + threadIdx.x) & ~31ull;   // first block of this warp
    const uint64_t b = b0 + lane;
    if (b0 >= nblocks) return;                                   // whole warp
    const uint32_t tp = tau_pattern<DT>(pfx_tau(tau_host, tau_from));
    const bool live = b < nblocks;
    // this lane's stream: next word and one past its last word, counted from the warp's first word
    // (32 blocks are at most 32 x 2176 words long: 32 bits do)
    const unsigned long long w0 = off[b0];
    const uint32_t *base = stream + w0;
    uint32_t at = 0u, end = 0u;
    if (live) { at = (uint32_t)(off[b] - w0); end = (uint32_t)(off[b + 1] - w0); }
    uint32_t bit = 0u;                                           // bits of word `at` already consumed
    const uint64_t i0 = b * LGN_PREFIX_BLOCK;
    const uint64_t i1 = !live ? i0 : (i0 + LGN_PREFIX_BLOCK < n ? i0 + LGN_PREFIX_BLOCK : n);
    for (uint32_t j = 0; j < LGN_PREFIX_BLOCK; j += 32) {
        // 1. rows: lane l fetches word l (and 32 + l) of every stream in turn
        {
            uint32_t first[32], more[32];                        // all 64 loads in flight together
            #pragma unroll
            for (int r = 0; r < 32; ++r) {
                const uint32_t ra = __shfl_sync(0xFFFFFFFFu, at, r) + lane, re = __shfl_sync(0xFFFFFFFFu, end, r);
                first[r] = ra < re ? __ldg(base + ra) : 0u;
                more[r] = (lane < kDecRowWords - 32 && ra + 32u < re) ? __ldg(base + ra + 32u) : 0u;
            }
            #pragma unroll
            for (int r = 0; r < 32; ++r) {
                rows[warp][r][lane] = first[r];
                if (lane < kDecRowWords - 32) rows[warp][r][32 + lane] = more[r];
            }
        }
        __syncwarp();
        // 2. decode
        const uint64_t ic = i0 + j;
        const uint32_t cnt = ic >= i1 ? 0u : (i1 - ic < 32u ? (uint32_t)(i1 - ic) : 32u);
        const uint32_t *row = rows[warp][lane];
        uint32_t pos = bit;
        #pragma unroll 4
        for (uint32_t k = 0; k < 32u; ++k) {
            const uint32_t wi = pos >> 5, sh = pos & 31u;
            const uint32_t a = row[wi], c = row[wi + 1], d = DT == LGN_F32 ? row[wi + 2] : 0u;  // bf16: 18 bits from bit 31 at most
            const uint32_t lo = __funnelshift_r(a, c, sh), hi = __funnelshift_r(c, d, sh);     // 64 bits from the current bit
            const uint32_t val = __funnelshift_r(lo, hi, 2) & (DT == LGN_F32 ? 0xFFFFFFFFu : 0xFFFFu);
            const bool nz = (lo & 1u) != 0u, isval = (lo & 2u) != 0u;
            const uint32_t alpha = (lo & 4u) ? (tp | PfxTraits<DT>::kSign) : tp;
            const uint32_t pat = nz ? (isval ? val : alpha) : 0u;
            const uint32_t len = nz ? (isval ? 2u + W : 3u) : 1u;
            if (k < cnt) { tile[warp][lane][k] = pat; pos += len; }
        }
        at += pos >> 5;
        bit = pos & 31u;
        __syncwarp();
        // 3. rows of elements out
        #pragma unroll 4
        for (int r = 0; r < 32; ++r) {                           // row r = block b0 + r, elements j .. j+31
            const uint64_t i = (b0 + r) * LGN_PREFIX_BLOCK + j + lane;
            if (b0 + r < nblocks && i < n) {
                const uint32_t v = tile[warp][r][lane];
                if (DT == LGN_F32) static_cast<uint32_t *>(out)[i] = v;
                else               static_cast<uint16_t *>(out)[i] = (uint16_t)v;
            }
        }
        __syncwarp();
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
    return (size_t)(sizeof(PfxCtl) + (lgn_prefix_blocks(n) * 8 + 255) / 256 * 256);
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
    const float tau_used = dt == LGN_BF16 ? snap_threshold_bf16(tau) : snap_threshold_f32(tau);
    const Weyl wy = { kWeyl0, kWeyl1 };
    if (nb == 0) {
        prefix_empty_kernel<<<1, 1, 0, st>>>(off_dev);
        return cudaGetLastError() == cudaSuccess ? LGN_OK : LGN_ERR_CUDA;
    }
    // ticket, error flag and the per-block look-back states start at zero
    if (cudaMemsetAsync(ws, 0, lgn_prefix_workspace_bytes(n), st) != cudaSuccess) return LGN_ERR_CUDA;
    PfxCtl *ctl = static_cast<PfxCtl *>(ws);
    unsigned long long *state = reinterpret_cast<unsigned long long *>(static_cast<char *>(ws) + sizeof(PfxCtl));
    #define LGN_PFX1(D, P) { const unsigned grid = resident_grid(prefix_encode_kernel<D, P>, nb); \
                             if (grid == 0) return LGN_ERR_CUDA; \
                             log_line("prefix encoder: %llu blocks of %u elements, grid %u x %d threads, Eq. 5 %s, threshold from %s", \
                                      (unsigned long long)nb, (unsigned)LGN_PREFIX_BLOCK, grid, kPfxThreads, P ? "applied" : "not applied", \
                                      tau_from_dev ? "a result record on the device" : "the host"); \
                             prefix_encode_kernel<D, P><<<grid, kPfxThreads, 0, st>>>(g, n, nb, tau_used, tau_from_dev, seed, wy, \
                                 ctl, state, off_dev, stream_dev, capacity_words); }
    if (dt == LGN_F32) { if (apply_prune) LGN_PFX1(LGN_F32, true) else LGN_PFX1(LGN_F32, false) }
    else               { if (apply_prune) LGN_PFX1(LGN_BF16, true) else LGN_PFX1(LGN_BF16, false) }
    #undef LGN_PFX1
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
    const unsigned grid = (unsigned)((nb + kDecThreads - 1) / kDecThreads);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dt == LGN_F32) prefix_decode_kernel<LGN_F32><<<grid, kDecThreads, 0, st>>>(stream_dev, off_dev, n, nb, tau_used, tau_from_dev, out_dev);
    else               prefix_decode_kernel<LGN_BF16><<<grid, kDecThreads, 0, st>>>(stream_dev, off_dev, n, nb, tau_used, tau_from_dev, out_dev);
    return cudaGetLastError() == cudaSuccess ? LGN_OK : LGN_ERR_CUDA;
}
