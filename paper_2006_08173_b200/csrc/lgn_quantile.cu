// Exact order statistic of |g| over the nonzero elements (the high quantile that
// estimates the cut k of a truncated lognormal; appendix "Neural gradients lognormal
// distributions are truncated", which takes a high quantile of the data, 0.997 as its
// example, for the cut).
//
// Magnitude patterns of IEEE values order like the values, so the element of rank r
// is found by radix selection on the pattern:
//   top    histogram of the upper 15 magnitude bits (the whole bf16 magnitude; bits
//          30..16 of an fp32 one) in shared memory, merged into global memory
//   pick   one CTA scans the 32768 counts: nnz, r = ceil(q nnz), the bin that holds
//          rank r and the rank inside it      -- bf16: that bin IS the value
//   low    fp32 only: histogram of the lower 16 bits of the elements in that bin
//          (global atomics: about one element in a thousand takes part)
//   pick   one CTA scans the 65536 counts -> the full pattern
// One read of a bf16 tensor, two of an fp32 tensor.
#include <cstring>

#include <cuda_runtime.h>

#include "lgn.h"
#include "lgn_device.cuh"

namespace lgn {

constexpr int kQTopBins = 1 << 15, kQLowBins = 1 << 16;
constexpr int kQThreads = 1024;
constexpr int kQInFlight = 4;                       // 32-byte chunks a thread loads before it uses the first

struct QCtl {
    unsigned long long nnz;
    unsigned long long rank_in_bin;                 // 1-based rank of the wanted element among its top bin's elements
    uint32_t           bin;                         // upper 15 magnitude bits of the wanted element
    uint32_t           pad[59];
};
static_assert(sizeof(QCtl) == 256, "control block");

constexpr size_t kQWsBytes = sizeof(QCtl) + sizeof(uint32_t) * (size_t)(kQTopBins + kQLowBins);

template <int DT>
__device__ __forceinline__ uint32_t magnitude(const Chunk &c, int e) {
    if (DT == LGN_F32) return c.w[e] & 0x7FFFFFFFu;
    return ((c.w[e >> 1] >> ((e & 1) * 16)) & 0x7FFFu) << 16;            // widened: the same 31-bit scale as fp32
}

// Walk over the tensor, kQInFlight chunks per thread per step; f(magnitude) for every element in range.
template <int DT, class F>
__device__ __forceinline__ void for_each_magnitude(const void *g, uint64_t n, F f) {
    constexpr int C = ElemTraits<DT>::kChunk;
    const uint64_t nchunks = (n + C - 1) / C;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t c0 = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; c0 < nchunks; c0 += stride * kQInFlight) {
        Chunk v[kQInFlight];
        #pragma unroll
        for (int j = 0; j < kQInFlight; ++j) {
            const uint64_t c = c0 + (uint64_t)j * stride;
            if (c < nchunks) v[j] = load_chunk<DT, false, Ld::Keep>(g, c * C, n);     // past n: zeros
            else { for (int k = 0; k < 8; ++k) v[j].w[k] = 0u; }
        }
        #pragma unroll
        for (int j = 0; j < kQInFlight; ++j) {
            #pragma unroll
            for (int e = 0; e < C; ++e) f(magnitude<DT>(v[j], e));
        }
    }
}

template <int DT>
__global__ void __launch_bounds__(kQThreads)
quantile_top_kernel(const void *g, uint64_t n, uint32_t *hist_top) {
    extern __shared__ uint32_t sh[];
    for (int k = threadIdx.x; k < kQTopBins; k += kQThreads) sh[k] = 0u;
    __syncthreads();
    for_each_magnitude<DT>(g, n, [&](uint32_t m) { if (m) atomicAdd(&sh[m >> 16], 1u); });
    __syncthreads();
    for (int k = threadIdx.x; k < kQTopBins; k += kQThreads) { const uint32_t c = sh[k]; if (c) atomicAdd(&hist_top[k], c); }
}

// Exclusive scan over the CTA of one value per thread; returns the exclusive prefix, *total = sum.
__device__ __forceinline__ unsigned long long cta_exclusive_scan(unsigned long long v, unsigned long long *sm /* 32 */,
                                                                 unsigned long long *total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long incl = v;
    #pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, incl, d); if (lane >= d) incl += t; }
    __syncthreads();
    if (lane == 31) sm[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        unsigned long long w = sm[lane];
        #pragma unroll
        for (int d = 1; d < 32; d <<= 1) { const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, w, d); if (lane >= d) w += t; }
        sm[lane] = w;
    }
    __syncthreads();
    *total = sm[31];
    return incl - v + (warp ? sm[warp - 1] : 0ull);
}

// Sum of the PER consecutive counts a thread owns, with 16-byte loads (all in flight together).
template <int PER>
__device__ __forceinline__ unsigned long long own_sum(const uint32_t *hist) {
    const uint4 *p = reinterpret_cast<const uint4 *>(hist + (size_t)threadIdx.x * PER);
    unsigned long long s = 0;
    #pragma unroll
    for (int k = 0; k < PER / 4; ++k) { const uint4 v = p[k]; s += (unsigned long long)v.x + v.y + v.z + v.w; }
    return s;
}

// Finds the bin that holds rank `rank` (1-based, 1 <= rank <= total): the thread whose PER
// bins contain it announces itself, then warp 0 scans those bins 32 at a time.  Returns
// true in one lane of warp 0, with *bin and *rank_in_bin set.  All threads must call.
template <int PER>
__device__ __forceinline__ bool locate(const uint32_t *hist, unsigned long long rank, unsigned long long mine,
                                       unsigned long long before, uint32_t *bin, unsigned long long *rank_in_bin) {
    __shared__ uint32_t sm_owner;
    __shared__ unsigned long long sm_before;
    if (rank > before && rank <= before + mine) { sm_owner = threadIdx.x; sm_before = before; }
    __syncthreads();
    if (threadIdx.x >= 32) return false;
    const int lane = threadIdx.x;
    const uint32_t base = sm_owner * PER;
    unsigned long long cum = sm_before;
    for (int j = 0; j < PER; j += 32) {
        const uint32_t c = hist[base + j + lane];
        unsigned long long incl = c;
        #pragma unroll
        for (int d = 1; d < 32; d <<= 1) { const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, incl, d); if (lane >= d) incl += t; }
        const bool hit = rank > cum + incl - c && rank <= cum + incl;
        if (__any_sync(0xFFFFFFFFu, hit)) {
            if (hit) { *bin = base + j + lane; *rank_in_bin = rank - (cum + incl - c); }
            return hit;
        }
        cum += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
    return false;
}

template <int DT>
__global__ void __launch_bounds__(kQThreads)
quantile_pick_top_kernel(const uint32_t *hist_top, double q, QCtl *ctl, lgn_quantile_t *out) {
    __shared__ unsigned long long sm[32];
    constexpr int PER = kQTopBins / kQThreads;
    unsigned long long nnz;
    const unsigned long long mine = own_sum<PER>(hist_top);
    const unsigned long long before = cta_exclusive_scan(mine, sm, &nnz);
    if (nnz == 0) {
        if (threadIdx.x == 0) { ctl->nnz = 0; ctl->rank_in_bin = 0; ctl->bin = 0; out->value = 0.f; out->pad = 0; out->nnz = 0; }
        return;
    }
    unsigned long long r = (unsigned long long)ceil(q * (double)nnz);
    if (r < 1) r = 1;
    if (r > nnz) r = nnz;
    uint32_t bin;
    unsigned long long rib;
    if (locate<PER>(hist_top, r, mine, before, &bin, &rib)) {
        ctl->nnz = nnz; ctl->bin = bin; ctl->rank_in_bin = rib;
        if (DT == LGN_BF16) { out->value = u2f(bin << 16); out->pad = 0; out->nnz = nnz; }
    }
}

__global__ void __launch_bounds__(kQThreads)
quantile_low_kernel(const void *g, uint64_t n, const QCtl *ctl, uint32_t *hist_low) {
    if (ctl->nnz == 0) return;
    const uint32_t bin = ctl->bin;
    for_each_magnitude<LGN_F32>(g, n, [&](uint32_t m) { if (m && (m >> 16) == bin) atomicAdd(&hist_low[m & 0xFFFFu], 1u); });
}

__global__ void __launch_bounds__(kQThreads)
quantile_pick_low_kernel(const uint32_t *hist_low, const QCtl *ctl, lgn_quantile_t *out) {
    __shared__ unsigned long long sm[32];
    if (ctl->nnz == 0) return;
    constexpr int PER = kQLowBins / kQThreads;
    unsigned long long total;
    const unsigned long long mine = own_sum<PER>(hist_low);
    const unsigned long long before = cta_exclusive_scan(mine, sm, &total);
    uint32_t low;
    unsigned long long rib;
    if (locate<PER>(hist_low, ctl->rank_in_bin, mine, before, &low, &rib)) {
        out->value = u2f((ctl->bin << 16) | low); out->pad = 0; out->nnz = ctl->nnz;
    }
}

}  // namespace lgn

using namespace lgn;

extern "C" size_t lgn_quantile_workspace_bytes(void) { return kQWsBytes; }

extern "C" lgn_status lgn_quantile(const void *g, uint64_t n, lgn_dtype dt, double q, lgn_quantile_t *out_dev,
                                   void *ws, size_t ws_bytes, void *stream) {
    if (dt != LGN_F32 && dt != LGN_BF16) return LGN_ERR_INVALID_ARG;
    if (!(q >= 0.0 && q <= 1.0)) return LGN_ERR_INVALID_ARG;
    if (out_dev == nullptr || (reinterpret_cast<uintptr_t>(out_dev) & 15u)) return LGN_ERR_INVALID_ARG;
    if (n > 0 && (g == nullptr || (reinterpret_cast<uintptr_t>(g) & 31u))) return LGN_ERR_INVALID_ARG;
    if (n >= (1ull << 32)) return LGN_ERR_UNSUPPORTED;       // the histogram bins count in 32 bits
    if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & 15u)) return LGN_ERR_INVALID_ARG;
    if (ws_bytes < kQWsBytes) return LGN_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    QCtl *ctl = static_cast<QCtl *>(ws);
    uint32_t *hist_top = reinterpret_cast<uint32_t *>(static_cast<char *>(ws) + sizeof(QCtl));
    uint32_t *hist_low = hist_top + kQTopBins;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return LGN_ERR_CUDA;
    const size_t smem = sizeof(uint32_t) * (size_t)kQTopBins;
    const void *top = dt == LGN_F32 ? reinterpret_cast<const void *>(&quantile_top_kernel<LGN_F32>)
                                    : reinterpret_cast<const void *>(&quantile_top_kernel<LGN_BF16>);
    if (cudaFuncSetAttribute(top, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return LGN_ERR_CUDA;
    if (cudaMemsetAsync(ws, 0, kQWsBytes, st) != cudaSuccess) return LGN_ERR_CUDA;
    const unsigned chunk = dt == LGN_F32 ? 8u : 16u;
    const uint64_t nchunks = (n + chunk - 1) / chunk;
    uint64_t want = (nchunks + (uint64_t)kQThreads * kQInFlight - 1) / ((uint64_t)kQThreads * kQInFlight);
    const unsigned grid = (unsigned)(want < 1 ? 1 : (want > (uint64_t)sms ? (uint64_t)sms : want));
    if (dt == LGN_F32) {
        quantile_top_kernel<LGN_F32><<<grid, kQThreads, smem, st>>>(g, n, hist_top);
        quantile_pick_top_kernel<LGN_F32><<<1, kQThreads, 0, st>>>(hist_top, q, ctl, out_dev);
        quantile_low_kernel<<<grid, kQThreads, 0, st>>>(g, n, ctl, hist_low);
        quantile_pick_low_kernel<<<1, kQThreads, 0, st>>>(hist_low, ctl, out_dev);
    } else {
        quantile_top_kernel<LGN_BF16><<<grid, kQThreads, smem, st>>>(g, n, hist_top);
        quantile_pick_top_kernel<LGN_BF16><<<1, kQThreads, 0, st>>>(hist_top, q, ctl, out_dev);
    }
    return cudaGetLastError() == cudaSuccess ? LGN_OK : LGN_ERR_CUDA;
}
