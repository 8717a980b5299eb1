// Decoder of packed FP codes: the last step of Algorithm 1, X_Q = 2^e_s * Q_FP(.),
// for the consumer of a quantised gradient (the following backward GEMM reads
// fp32 or bf16).
//
// A code [sign | exponent field f | mantissa m] with f != 0 stands for
// (-1)^s (1 + m 2^-n1) 2^(f - E_max + e_s)  (Eq. 1-2), which is the fp32 pattern
//     sign << 31 | (f + K) << 23 | m << (23 - n1),      K = 127 + e_s - E_max,
// i.e. the integer [f | m] shifted left by 23 - n1 plus K << 23: one multiply-add.
// f == 0 is zero.  The host accepts a format only if every f + K is a normal fp32
// exponent (1..254), so no decoded value is subnormal, infinite or rounded; bf16
// output is the upper half of the same pattern (n1 <= 6 < 7 fraction bits).
//
// One CTA handles tiles of kDqTileElems elements: the tile's code words (a whole
// number of 32-bit words for every width) are brought into shared memory with
// coalesced loads, then thread t decodes the t-th 32-byte chunk of each 8 KiB
// span of the output, so every warp store covers 1 KiB of contiguous memory.
#include <cstring>

#include <cuda_runtime.h>

#include "lgn.h"
#include "lgn_device.cuh"

namespace lgn {

constexpr int kDqTileElems = 8192;

struct DequantParams {
    uint32_t mult;       // 2^(23 - man_bits): places [field | mantissa] in an fp32 pattern
    uint32_t k23;        // K << 23
    uint32_t min_code;   // 2^man_bits: magnitudes below it have exponent field 0
};

// fp32 pattern of the code whose bit 0 is bit `pos` of the little-endian word
// sequence v[] (pos is a compile-time constant once the loops are unrolled).
template <int NBITS>
__device__ __forceinline__ uint32_t decode_at(const uint32_t *v, int pos, const DequantParams &p) {
    const int k = pos >> 5, s = pos & 31;
    const uint32_t raw = (s + NBITS <= 32) ? (v[k] >> s) : __funnelshift_r(v[k], v[k + 1], s);   // bits above NBITS: junk
    const uint32_t mag = raw & ((1u << (NBITS - 1)) - 1u);
    const uint32_t body = (mag * p.mult + p.k23) | ((raw << (32 - NBITS)) & 0x80000000u);
    return mag >= p.min_code ? body : 0u;                        // exponent field 0: +0 whatever the other bits
}

template <int NBITS, int ODT>
__global__ void __launch_bounds__(kThreads)
dequantize_kernel(const uint32_t *__restrict__ codes, void *__restrict__ out, uint64_t n, uint64_t total_words,
                  uint32_t ntiles, const DequantParams p) {
    constexpr int C = ElemTraits<ODT>::kChunk;                  // output elements per 32-byte chunk
    constexpr int kTileWords = kDqTileElems * NBITS / 32;       // 256 * NBITS
    constexpr int kChunksPerThread = kDqTileElems / (C * kThreads);
    constexpr int kChunkBits = C * NBITS;
    constexpr int NW = (kChunkBits + 31) / 32;                  // words that hold a chunk's codes once aligned
    __shared__ uint32_t sm[kTileWords + 4];                     // + words a chunk's window may reach past the tile

    // the next tile's code words are fetched into registers while the current tile is decoded
    uint32_t r_next[NBITS];
    auto fetch = [&](uint32_t tile) {
        const uint64_t w0 = (uint64_t)tile * kTileWords;
        #pragma unroll
        for (int k = 0; k < NBITS; ++k) {
            const uint64_t w = w0 + (uint64_t)(k * kThreads + threadIdx.x);
            r_next[k] = (tile < ntiles && w < total_words) ? __ldcs(codes + w) : 0u;
        }
    };
    fetch(blockIdx.x);
    for (uint32_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        __syncthreads();                                        // the previous tile has been decoded
        #pragma unroll
        for (int k = 0; k < NBITS; ++k) sm[k * kThreads + threadIdx.x] = r_next[k];
        if (threadIdx.x < 4) sm[kTileWords + threadIdx.x] = 0u;
        __syncthreads();
        fetch(tile + gridDim.x);

        const uint64_t tile_base = (uint64_t)tile * kDqTileElems;
        const bool full = tile_base + kDqTileElems <= n;
        #pragma unroll
        for (int j = 0; j < kChunksPerThread; ++j) {
            const int chunk = j * kThreads + threadIdx.x;
            const uint64_t i = tile_base + (uint64_t)chunk * C;
            if (!full && i >= n) continue;
            const int byte0 = chunk * (kChunkBits / 8);         // C*NBITS is a multiple of 8
            const int sh = (byte0 & 3) * 8;
            uint32_t r[NW + 1], v[NW + 1];
            #pragma unroll
            for (int k = 0; k <= NW; ++k) r[k] = sm[(byte0 >> 2) + k];
            #pragma unroll
            for (int k = 0; k < NW; ++k) v[k] = __funnelshift_r(r[k], r[k + 1], sh);
            v[NW] = 0u;
            Chunk o;
            if constexpr (ODT == LGN_F32) {
                #pragma unroll
                for (int e = 0; e < C; ++e) o.w[e] = decode_at<NBITS>(v, e * NBITS, p);
            } else {
                #pragma unroll
                for (int e = 0; e < C; e += 2) {                 // the upper halves of two fp32 patterns: one byte permute
                    const uint32_t b0 = decode_at<NBITS>(v, e * NBITS, p), b1 = decode_at<NBITS>(v, (e + 1) * NBITS, p);
                    o.w[e >> 1] = __byte_perm(b0, b1, 0x7632);
                }
            }
            if (full) store_chunk<ODT, true>(out, i, n, o);
            else      store_chunk<ODT, false>(out, i, n, o);
        }
    }
}

#define LGN_DK(NB, DT) reinterpret_cast<const void *>(&dequantize_kernel<NB, DT>)
static const void *const kDequantTable[2][5] = {
    { LGN_DK(4, LGN_F32), LGN_DK(5, LGN_F32), LGN_DK(6, LGN_F32), LGN_DK(7, LGN_F32), LGN_DK(8, LGN_F32) },
    { LGN_DK(4, LGN_BF16), LGN_DK(5, LGN_BF16), LGN_DK(6, LGN_BF16), LGN_DK(7, LGN_BF16), LGN_DK(8, LGN_BF16) } };
#undef LGN_DK

}  // namespace lgn

using namespace lgn;

extern "C" lgn_status lgn_dequantize(const void *codes, uint64_t n, const lgn_fp_format_t *fmt, lgn_dtype out_dt,
                                     void *out, void *stream) {
    if (fmt == nullptr) return LGN_ERR_INVALID_ARG;
    if (fmt->nbits < 4 || fmt->nbits > 8) return LGN_ERR_UNSUPPORTED;
    if (fmt->exp_bits < 1 || fmt->man_bits < 0 || 1 + fmt->exp_bits + fmt->man_bits != fmt->nbits)
        return LGN_ERR_INVALID_ARG;
    if (out_dt != LGN_F32 && out_dt != LGN_BF16) return LGN_ERR_INVALID_ARG;
    if (fmt->scale_exp < -400 || fmt->scale_exp > 400) return LGN_ERR_INVALID_ARG;
    const int Emax = 1 << (fmt->exp_bits - 1);
    const int K = 127 + fmt->scale_exp - Emax;
    if (K < 0 || K + (1 << fmt->exp_bits) - 1 > 254) return LGN_ERR_UNSUPPORTED;   // a code outside the normal fp32 range
    if (n > (1ull << 44)) return LGN_ERR_UNSUPPORTED;
    if (n == 0) return LGN_OK;
    if (codes == nullptr || out == nullptr) return LGN_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(codes) & 15u) || (reinterpret_cast<uintptr_t>(out) & 31u)) return LGN_ERR_INVALID_ARG;
    {
        const size_t cb = lgn_codes_bytes(n, fmt->nbits), ob = (size_t)n * (out_dt == LGN_BF16 ? 2u : 4u);
        const char *a = static_cast<const char *>(codes), *b = static_cast<const char *>(out);
        if (a < b + ob && b < a + cb) return LGN_ERR_INVALID_ARG;                  // overlap
    }
    const void *fn = kDequantTable[out_dt][fmt->nbits - 4];
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kThreads, 0) != cudaSuccess)
        return LGN_ERR_CUDA;
    if (per_sm < 1) per_sm = 1;
    uint32_t ntiles = (uint32_t)((n + kDqTileElems - 1) / kDqTileElems);
    unsigned grid = (unsigned)(sms * per_sm);
    if (grid > ntiles) grid = ntiles;
    uint64_t total_words = (n * (uint64_t)fmt->nbits + 31) >> 5;
    DequantParams p;
    p.mult = 1u << (23 - fmt->man_bits);
    p.k23 = (uint32_t)K << 23;
    p.min_code = 1u << fmt->man_bits;
    void *args[] = { &codes, &out, &n, &total_words, &ntiles, &p };
    if (cudaLaunchKernel(fn, dim3(grid), dim3(kThreads), args, 0, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return LGN_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? LGN_OK : LGN_ERR_CUDA;
}
