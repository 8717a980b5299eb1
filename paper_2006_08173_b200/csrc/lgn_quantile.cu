// Exact order statistic of |g| over the nonzero elements (the high quantile that
// estimates the cut k of a truncated lognormal; appendix "Neural gradients lognormal
// distributions are truncated", which takes a high quantile of the data, 0.997 as its
// example, for the cut).
//
// Magnitude patterns of IEEE values order like the values, so the element of rank r
// is found by selection on the pattern.  Two ways:
//
// The "histogram path" (radix selection):
//   top    histogram of the upper 15 magnitude bits (the whole bf16 magnitude; bits
//          30..16 of an fp32 one) in shared memory, merged into global memory; the CTA
//          that finishes last scans the 32768 counts: nnz, r = ceil(q nnz), the bin that
//          holds rank r and the rank inside it      -- bf16: that bin IS the value
//   low    fp32 only: histogram of the lower 16 bits of the elements in that bin
//          (global atomics: about one element in a thousand takes part); the last CTA
//          scans the 65536 counts -> the full pattern
// One read of a bf16 tensor, two of an fp32 tensor, each bound by the shared-memory
// atomics, one per element.
//
// The "bracket path", taken first by tensors of 2^24 elements and more, reads the tensor
// once, with no atomic on the way of an ordinary element:
//   sample   top histogram of a sample of 32-byte chunks spread over the tensor; the last
//            CTA takes the sample's order statistics a few standard errors below and above
//            rank q m (m = nonzero elements of the sample): pattern bounds [lo, hi), on
//            histogram-bin boundaries, that hold the wanted element
//   count    the full read: counts the nonzero elements and those >= lo in registers;
//            the few elements inside [lo, hi) are set aside (fp32: their patterns are
//            appended to one of 16 lists, by the leading bits of pattern - lo, staged
//            per CTA in shared memory; bf16: counted per value in a small shared-memory
//            histogram).  The last CTA finishes: nnz and
//            the rank r are now exact; if the elements below lo number less than r and
//            those below hi at least r, the element of rank r - below among those set
//            aside is the answer (fp32: the lists' lengths tell which list holds it, then
//            radix selection over that list, 12 bits a pass; bf16: a scan of the
//            bracket's bins).  Otherwise (an unrepresentative sample,
//            a list that overflowed) it raises `fallback`, and the histogram path's
//            kernels, launched behind it, do the work instead of returning at once.
// The result is exact either way.
#include <cmath>
#include <cstring>

#include <cuda_runtime.h>

#include "lgn.h"
#include "lgn_device.cuh"
#include "lgn_log.h"

namespace lgn {

constexpr int kQTopBins = 1 << 15, kQLowBins = 1 << 16;
constexpr int kQThreads = 1024;
constexpr int kQInFlight = 4;                       // 32-byte chunks a thread loads before it uses the first
constexpr uint64_t kQDirect = 1ull << 24;           // below this: the histogram path at once
constexpr uint32_t kQSampleMin = 1u << 21;          // elements in the sample, at least
constexpr double   kQSigmas = 8.0;                  // half-width of the bracket in standard errors of the sample's rank
constexpr uint32_t kQListCap = 1u << 20;            // fp32 patterns the count pass may set aside (4 MiB),
constexpr int kQBuckets = 16;                       // in this many lists by the leading bits of (pattern - lo)
constexpr uint32_t kQBucketCap = kQListCap / kQBuckets;
constexpr int kQCountThreads = 512;
constexpr int kQRoundSteps = 2;                     // a round of the count pass: this many steps of kQInFlight chunks per thread (128 KiB)
constexpr int kQCoarse = 128;                       // groups of 256 bins whose sums the sample pass also keeps
constexpr int kQSideBins = 4096;                    // fp32: patterns staged per CTA; bf16: values a bracket may span;
                                                    // also the bins of one radix pass over the list

struct QCtl {
    unsigned long long nnz;                         // histogram path: set by top's scan
    unsigned long long rank_in_bin;                 // 1-based rank of the wanted element among its top bin's elements
    uint32_t           bin;                         // upper 15 magnitude bits of the wanted element
    // bracket path
    uint32_t           lo;                          // first pattern of the bracket (>= 1: a zero is never inside)
    uint32_t           width;                       // hi - lo
    uint32_t           fallback;                    // set by count's finish: the histogram path has to run
    unsigned long long count_nz;                    // nonzero elements
    unsigned long long count_ge;                    // elements with pattern >= lo
    uint32_t           ticket[4];                   // CTAs done, per kernel (sample, count, top, low)
    uint32_t           next_round;                  // count pass: rounds handed out
    uint32_t           bucket[kQBuckets];           // fp32: patterns set aside per list (may pass kQBucketCap: then that list is short)
    uint32_t           pad[31];
};
static_assert(sizeof(QCtl) == 256, "control block");

// Workspace: [control | top bins | low bins (bf16: the bracket's bins) | the sample's top bins | their group sums | list]
constexpr size_t kQZeroedBytes = sizeof(QCtl) + sizeof(uint32_t) * (size_t)(kQTopBins + kQLowBins + kQTopBins + kQCoarse);   // cleared per call
constexpr size_t kQWsBytes = kQZeroedBytes + sizeof(uint32_t) * (size_t)kQListCap;

// Launch order inside one call: every kernel but the first is launched with programmatic
// stream serialisation, lets its successor become resident at once and waits for its
// predecessor's results before it touches them.
__device__ __forceinline__ void let_successor_in() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void wait_for_predecessor() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

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

// ---------------------------------------------------------------- one-CTA steps
// All of them are run by the CTA that finishes a kernel last, on what the other CTAs
// left in global memory: its reads go to L2 (ld.cg).

// True in every thread of exactly one CTA: the one whose ticket is the last.  Every
// thread's global writes and atomics precede the ticket; the caller's reads follow it.
__device__ __forceinline__ bool last_cta_done(uint32_t *ticket) {
    __shared__ uint32_t sm_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) sm_last = atomicAdd(ticket, 1u) == gridDim.x - 1u;
    __syncthreads();
    const bool last = sm_last != 0u;
    if (last) __threadfence();
    return last;
}

// Exclusive scan over the CTA of one value per thread; returns the exclusive prefix, *total = sum.
__device__ __forceinline__ unsigned long long cta_exclusive_scan(unsigned long long v, unsigned long long *sm /* 32 */,
                                                                 unsigned long long *total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
    unsigned long long incl = v;
    #pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, incl, d); if (lane >= d) incl += t; }
    __syncthreads();
    if (lane == 31) sm[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        unsigned long long w = lane < warps ? sm[lane] : 0ull;
        #pragma unroll
        for (int d = 1; d < 32; d <<= 1) { const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, w, d); if (lane >= d) w += t; }
        sm[lane] = w;
    }
    __syncthreads();
    *total = sm[31];
    return incl - v + (warp ? sm[warp - 1] : 0ull);
}

// Sum of the PER consecutive counts a thread owns, with 16-byte loads (all in flight together).
// SHARED: the counts are in this CTA's shared memory.
template <int PER, bool SHARED>
__device__ __forceinline__ unsigned long long own_sum(const uint32_t *hist) {
    const uint4 *p = reinterpret_cast<const uint4 *>(hist + (size_t)threadIdx.x * PER);
    unsigned long long s = 0;
    #pragma unroll
    for (int k = 0; k < PER / 4; ++k) { const uint4 v = SHARED ? p[k] : __ldcg(p + k); s += (unsigned long long)v.x + v.y + v.z + v.w; }
    return s;
}

// Finds the bins that hold the ranks rank[0] and rank[1] (1-based, 1 <= rank <= total; 0: none
// wanted): the thread whose PER bins contain a rank announces itself, then warp w scans the bins
// of rank[w]'s owner, 32 at a time.  The answers come back in every thread (through shared
// memory).  All threads must call.
template <int PER, bool SHARED>
__device__ __forceinline__ void locate_pair(const uint32_t *hist, const unsigned long long (&rank)[2], unsigned long long mine,
                                            unsigned long long before, uint32_t (&bin)[2], unsigned long long (&rank_in_bin)[2]) {
    __shared__ uint32_t sm_owner[2], sm_bin[2];
    __shared__ unsigned long long sm_before[2], sm_rib[2];
    __syncthreads();                                       // the previous call's answers have been read
    #pragma unroll
    for (int w = 0; w < 2; ++w)
        if (rank[w] > before && rank[w] <= before + mine) { sm_owner[w] = threadIdx.x; sm_before[w] = before; }
    __syncthreads();
    const int w = threadIdx.x >> 5;
    const unsigned long long want = w == 0 ? rank[0] : rank[1];
    if (w < 2 && want != 0ull) {
        const int lane = threadIdx.x & 31;
        const uint32_t base = sm_owner[w] * PER;
        unsigned long long cum = sm_before[w];
        constexpr int STEPS = (PER + 31) / 32;
        uint32_t counts[STEPS];
        #pragma unroll
        for (int s = 0; s < STEPS; ++s)                    // all in flight together
            counts[s] = s * 32 + lane < PER ? (SHARED ? hist[base + s * 32 + lane] : __ldcg(hist + base + s * 32 + lane)) : 0u;
        #pragma unroll
        for (int s = 0; s < STEPS; ++s) {
            const uint32_t c = counts[s];
            unsigned long long incl = c;
            #pragma unroll
            for (int d = 1; d < 32; d <<= 1) { const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, incl, d); if (lane >= d) incl += t; }
            const bool hit = c != 0u && want > cum + incl - c && want <= cum + incl;
            if (__any_sync(0xFFFFFFFFu, hit)) {
                if (hit) { sm_bin[w] = base + s * 32 + lane; sm_rib[w] = want - (cum + incl - c); }
                break;
            }
            cum += __shfl_sync(0xFFFFFFFFu, incl, 31);
        }
    }
    __syncthreads();
    #pragma unroll
    for (int k = 0; k < 2; ++k) { bin[k] = sm_bin[k]; rank_in_bin[k] = sm_rib[k]; }
}

template <int PER, bool SHARED>
__device__ __forceinline__ void locate(const uint32_t *hist, unsigned long long rank, unsigned long long mine,
                                       unsigned long long before, uint32_t *bin, unsigned long long *rank_in_bin) {
    const unsigned long long ranks[2] = { rank, 0ull };
    uint32_t bins[2];
    unsigned long long ribs[2];
    locate_pair<PER, SHARED>(hist, ranks, mine, before, bins, ribs);
    *bin = bins[0];
    *rank_in_bin = ribs[0];
}

// ---------------------------------------------------------------- histogram path

// `always` = 0: the kernel was launched behind the bracket path and works only if that gave up.
template <int DT>
__global__ void __launch_bounds__(kQThreads)
quantile_top_kernel(const void *g, uint64_t n, uint32_t *hist_top, double q, QCtl *ctl, lgn_quantile_t *out, int always) {
    extern __shared__ uint32_t sh[];
    __shared__ unsigned long long sm[32];
    let_successor_in();
    wait_for_predecessor();
    if (!always && __ldcg(&ctl->fallback) == 0u) return;    // ctl->nnz stays 0: the low kernel returns too
    for (int k = threadIdx.x; k < kQTopBins; k += kQThreads) sh[k] = 0u;
    __syncthreads();
    for_each_magnitude<DT>(g, n, [&](uint32_t m) { if (m) atomicAdd(&sh[m >> 16], 1u); });
    __syncthreads();
    for (int k = threadIdx.x; k < kQTopBins; k += kQThreads) { const uint32_t c = sh[k]; if (c) atomicAdd(&hist_top[k], c); }
    if (!last_cta_done(&ctl->ticket[2])) return;
    // the scan of the merged counts
    constexpr int PER = kQTopBins / kQThreads;
    unsigned long long nnz;
    const unsigned long long mine = own_sum<PER, false>(hist_top);
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
    locate<PER, false>(hist_top, r, mine, before, &bin, &rib);
    if (threadIdx.x == 0) {
        ctl->nnz = nnz; ctl->bin = bin; ctl->rank_in_bin = rib;
        if (DT == LGN_BF16) { out->value = u2f(bin << 16); out->pad = 0; out->nnz = nnz; }
    }
}

__global__ void __launch_bounds__(kQThreads)
quantile_low_kernel(const void *g, uint64_t n, QCtl *ctl, uint32_t *hist_low, lgn_quantile_t *out) {
    __shared__ unsigned long long sm[32];
    wait_for_predecessor();
    const unsigned long long nnz = __ldcg(&ctl->nnz);
    if (nnz == 0) return;
    const uint32_t bin = __ldcg(&ctl->bin);
    for_each_magnitude<LGN_F32>(g, n, [&](uint32_t m) { if (m && (m >> 16) == bin) atomicAdd(&hist_low[m & 0xFFFFu], 1u); });
    if (!last_cta_done(&ctl->ticket[3])) return;
    constexpr int PER = kQLowBins / kQThreads;
    unsigned long long total;
    const unsigned long long mine = own_sum<PER, false>(hist_low);
    const unsigned long long before = cta_exclusive_scan(mine, sm, &total);
    uint32_t low;
    unsigned long long rib;
    locate<PER, false>(hist_low, __ldcg(&ctl->rank_in_bin), mine, before, &low, &rib);
    if (threadIdx.x == 0) { out->value = u2f((bin << 16) | low); out->pad = 0; out->nnz = nnz; }
}

// ---------------------------------------------------------------- bracket path

__device__ __forceinline__ uint32_t mix32(uint32_t j) {
    uint32_t h = j * 0x9E3779B1u;
    h ^= h >> 16;
    return h * 0x9E3779B1u;
}

// Top histogram of `nsample` chunks: chunk j of the sample is taken from the j-th run
// of `step` consecutive chunks of the tensor, at a place inside the run that depends on
// j through a mixer (so that a period in the data does not meet a period in the sample).
// The last CTA turns it into the bracket.  m = nonzero elements of the sample; the wanted
// element has rank about q m in the sample, with a standard error of sqrt(m q (1 - q))
// ranks: the bracket runs from the bin of sample rank q m - kQSigmas errors to the bin of
// q m + kQSigmas errors (two ranks of slack on each side; open-ended where such a rank
// does not exist).  Next to the 32768 counts the CTAs keep the sums of groups of 256 bins,
// so that the last CTA reads 128 sums and two groups instead of every count.
template <int DT>
__global__ void __launch_bounds__(kQThreads)
quantile_sample_kernel(const void *g, uint64_t n, uint32_t nsample, uint32_t step, uint32_t *hist_sample, uint32_t *coarse,
                       double q, QCtl *ctl) {
    extern __shared__ uint32_t sh[];
    __shared__ unsigned long long sm[32];
    __shared__ uint32_t sm_coarse[kQCoarse];
    constexpr int C = ElemTraits<DT>::kChunk;
    let_successor_in();
    if (threadIdx.x < kQCoarse) sm_coarse[threadIdx.x] = 0u;
    for (int k = threadIdx.x; k < kQTopBins; k += kQThreads) sh[k] = 0u;
    __syncthreads();
    const uint32_t stride = gridDim.x * kQThreads;
    for (uint32_t j0 = blockIdx.x * kQThreads + threadIdx.x; j0 < nsample; j0 += 2u * stride) {
        Chunk v[2];
        #pragma unroll
        for (int k = 0; k < 2; ++k) {
            const uint32_t j = j0 + (uint32_t)k * stride;
            if (j < nsample) {
                const uint64_t c = (uint64_t)j * step + (((uint64_t)mix32(j) * step) >> 32);
                v[k] = load_chunk<DT, false, Ld::Keep>(g, c * C, n);
            } else {
                for (int e = 0; e < 8; ++e) v[k].w[e] = 0u;
            }
        }
        #pragma unroll
        for (int k = 0; k < 2; ++k) {
            #pragma unroll
            for (int e = 0; e < C; ++e) { const uint32_t m = magnitude<DT>(v[k], e); if (m) atomicAdd(&sh[m >> 16], 1u); }
        }
    }
    __syncthreads();
    // merge; bins k = thread + 1024 j: the 256 threads that share thread >> 8 hold one group per j
    #pragma unroll 4
    for (int j = 0; j < kQTopBins / kQThreads; ++j) {
        const int k = threadIdx.x + j * kQThreads;
        const uint32_t c = sh[k];
        if (c) atomicAdd(&hist_sample[k], c);
        const uint32_t w = __reduce_add_sync(0xFFFFFFFFu, c);
        if ((threadIdx.x & 31) == 0 && w) atomicAdd(&sm_coarse[k >> 8], w);
    }
    __syncthreads();
    if (threadIdx.x < kQCoarse && sm_coarse[threadIdx.x]) atomicAdd(&coarse[threadIdx.x], sm_coarse[threadIdx.x]);
    if (!last_cta_done(&ctl->ticket[0])) return;
    constexpr int PER = kQTopBins / kQCoarse;              // thread t < 128 owns group t
    unsigned long long m;
    const unsigned long long mine = threadIdx.x < kQCoarse ? (unsigned long long)__ldcg(coarse + threadIdx.x) : 0ull;
    const unsigned long long before = cta_exclusive_scan(mine, sm, &m);
    uint32_t lo = 1u, hi = 0x80000000u;
    if (m > 0) {                                           // uniform over the CTA
        const double centre = q * (double)m, dev = kQSigmas * sqrt((double)m * q * (1.0 - q)) + 2.0;
        const double r_lo = floor(centre - dev), r_hi = ceil(centre + dev);
        const unsigned long long ranks[2] = { r_lo >= 1.0 ? (unsigned long long)r_lo : 0ull, r_hi <= (double)m ? (unsigned long long)r_hi : 0ull };
        uint32_t bins[2];
        unsigned long long ribs[2];
        locate_pair<PER, false>(hist_sample, ranks, mine, before, bins, ribs);
        if (ranks[0]) { lo = bins[0] << 16; if (lo < 1u) lo = 1u; }
        if (ranks[1]) hi = (bins[1] + 1u) << 16;
    }
    if (threadIdx.x == 0) { ctl->lo = lo; ctl->width = hi - lo; }
}

// The full read.  Registers count the nonzero elements and those at or above lo; an
// element inside the bracket (rare) is set aside.  The tensor is handed out in rounds of
// 128 KiB through a counter, one round ahead (CTAs do not get equal shares of the memory
// system: with equal static shares the slowest finished 25 to 45 % after the first).  The
// last CTA finishes.
template <int DT>
__global__ void __launch_bounds__(kQCountThreads, 2)
quantile_count_kernel(const void *g, uint64_t n, double q, QCtl *ctl, uint32_t *list, uint32_t *hist_bracket, lgn_quantile_t *out) {
    constexpr int C = ElemTraits<DT>::kChunk;
    __shared__ __align__(16) uint32_t sm_side[kQSideBins];                // fp32: staged patterns; bf16: the bracket's bins
    __shared__ uint32_t sm_listed;
    __shared__ uint16_t sm_pos[DT == LGN_F32 ? kQSideBins : 1];           // a staged pattern's place among the CTA's patterns of its list
    __shared__ uint32_t sm_bcount[kQBuckets], sm_bbase[kQBuckets];
    __shared__ uint32_t sm_red[2][kQCountThreads / 32];
    __shared__ unsigned long long sm[32];
    __shared__ uint32_t sm_round[2];
    let_successor_in();
    if (DT == LGN_BF16) for (int k = threadIdx.x; k < kQSideBins; k += kQCountThreads) sm_side[k] = 0u;
    if (threadIdx.x == 0) sm_listed = 0u;
    wait_for_predecessor();
    const uint32_t lo = __ldcg(&ctl->lo), width = __ldcg(&ctl->width);
    const int bshift = width > (uint32_t)kQBuckets ? 32 - __clz(width - 1u) - 4 : 0;       // (pattern - lo) >> bshift < 16
    if (threadIdx.x == 0) sm_round[0] = atomicAdd(&ctl->next_round, 1u);
    __syncthreads();
    // bf16: both halves of a word at once, in 16-bit lanes.  With the sign bit of each lane forced to 1
    // a lane is 0x8000 + magnitude; minus a bound b <= 0x8000 it keeps bit 15 exactly when magnitude >= b.
    const uint32_t lo16 = (lo >> 16) < 1u ? 1u : (lo >> 16), hi16 = (lo + width) >> 16;       // bf16 patterns
    const uint32_t lo2 = lo16 * 0x00010001u, hi2 = hi16 * 0x00010001u;
    uint32_t nz = 0, ge = 0;                               // bf16: 0x8000 x the count, flushed every round
    uint32_t nz_total = 0, ge_total = 0;                   // a thread sees less than 2^32 elements (n < 2^32)
    auto set_aside = [&](uint32_t m) {                     // m: 31-bit pattern inside the bracket
        if (DT == LGN_F32) {
            const uint32_t slot = atomicAdd(&sm_listed, 1u);
            if (slot < (uint32_t)kQSideBins) sm_side[slot] = m;
            else {                                         // the CTA's stage is full: straight to its list
                const uint32_t b = (m - lo) >> bshift, at = atomicAdd(&ctl->bucket[b], 1u);
                if (at < kQBucketCap) list[b * kQBucketCap + at] = m;
            }
        } else {
            const uint32_t b = (m >> 16) - lo16;
            if (b < (uint32_t)kQSideBins) atomicAdd(&sm_side[b], 1u);          // a wider bracket is given up below
        }
    };
    auto take = [&](const Chunk &v) {
        if (DT == LGN_F32) {
            bool any = false;
            #pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint32_t m = v.w[e] & 0x7FFFFFFFu;
                nz_total += m != 0u;
                ge_total += m >= lo;
                any |= (m - lo) < width;
            }
            if (any) {
                #pragma unroll
                for (int e = 0; e < 8; ++e) { const uint32_t m = v.w[e] & 0x7FFFFFFFu; if ((m - lo) < width) set_aside(m); }
            }
        } else {
            uint32_t any = 0u;
            #pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint32_t b = v.w[e] | 0x80008000u;
                const uint32_t t1 = b - 0x00010001u, t = b - lo2, t2 = b - hi2;    // bit 15 of a lane: magnitude >= 1, >= lo, >= hi
                nz = __dp2a_lo(t1 & 0x80008000u, 0x0101u, nz);                // + 0x8000 per lane whose flag is set
                ge = __dp2a_lo(t & 0x80008000u, 0x0101u, ge);
                any |= t & ~t2;
            }
            if (any & 0x80008000u) {
                #pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const uint32_t m16 = (v.w[e >> 1] >> ((e & 1) * 16)) & 0x7FFFu;
                    if (m16 >= lo16 && m16 < hi16) set_aside(m16 << 16);
                }
            }
        }
    };
    auto flush_lanes = [&]() {
        if (DT == LGN_BF16) {
            nz_total += nz >> 15; ge_total += ge >> 15;
            nz = 0u; ge = 0u;
        }
    };
    const uint64_t nfull = n / C;                          // whole chunks
    constexpr uint32_t kStep = kQCountThreads * kQInFlight, kRound = kStep * kQRoundSteps;     // chunks
    const uint32_t nrounds = (uint32_t)((nfull + kRound - 1) / kRound);
    const char *base = static_cast<const char *>(g);
    for (uint32_t it = 0;; ++it) {
        const uint32_t round = sm_round[it & 1u];
        if (round >= nrounds) break;
        if (threadIdx.x == 0) sm_round[(it + 1u) & 1u] = atomicAdd(&ctl->next_round, 1u);     // its latency hides behind this round
        // two halves of kQInFlight / 2 chunks per thread: one is in flight while the other is counted
        constexpr int H = kQInFlight / 2, kHalves = 2 * kQRoundSteps;
        const uint64_t r0 = (uint64_t)round * kRound + threadIdx.x;
        auto fetch = [&](Chunk (&v)[H], int half) {
            #pragma unroll
            for (int j = 0; j < H; ++j) {
                const uint64_t c = r0 + (uint64_t)(half * H + j) * kQCountThreads;
                if (c < nfull) v[j] = ld32<Ld::Stream, true>(base + c * 32u);
                else { for (int k = 0; k < 8; ++k) v[j].w[k] = 0u; }
            }
        };
        Chunk va[H], vb[H];
        fetch(va, 0);
        #pragma unroll 1
        for (int h = 0; h < kHalves; h += 2) {
            fetch(vb, h + 1);
            #pragma unroll
            for (int j = 0; j < H; ++j) take(va[j]);
            if (h + 2 < kHalves) fetch(va, h + 2);
            #pragma unroll
            for (int j = 0; j < H; ++j) take(vb[j]);
        }
        flush_lanes();                                     // a round adds at most 256 x 0x8000
        if (round == 0 && threadIdx.x == 0 && nfull * C < n) take(load_chunk<DT, false, Ld::Keep>(g, nfull * C, n));
        __syncthreads();
    }
    flush_lanes();
    // CTA sums, one atomic per counter
    #pragma unroll
    for (int d = 16; d; d >>= 1) { nz_total += __shfl_xor_sync(0xFFFFFFFFu, nz_total, d); ge_total += __shfl_xor_sync(0xFFFFFFFFu, ge_total, d); }
    if ((threadIdx.x & 31) == 0) { sm_red[0][threadIdx.x >> 5] = nz_total; sm_red[1][threadIdx.x >> 5] = ge_total; }
    __syncthreads();                                       // also: every set_aside of the CTA is done
    if (threadIdx.x == 0) {
        unsigned long long a = 0, b = 0;
        for (int k = 0; k < kQCountThreads / 32; ++k) { a += sm_red[0][k]; b += sm_red[1][k]; }
        if (a) atomicAdd(&ctl->count_nz, a);
        if (b) atomicAdd(&ctl->count_ge, b);
    }
    if (DT == LGN_F32) {
        // the staged patterns go to their lists: one reservation per list and CTA
        const uint32_t staged = sm_listed < (uint32_t)kQSideBins ? sm_listed : (uint32_t)kQSideBins;
        if (threadIdx.x < kQBuckets) sm_bcount[threadIdx.x] = 0u;
        __syncthreads();
        for (uint32_t k = threadIdx.x; k < staged; k += kQCountThreads) sm_pos[k] = (uint16_t)atomicAdd(&sm_bcount[(sm_side[k] - lo) >> bshift], 1u);
        __syncthreads();
        if (threadIdx.x < kQBuckets && sm_bcount[threadIdx.x]) sm_bbase[threadIdx.x] = atomicAdd(&ctl->bucket[threadIdx.x], sm_bcount[threadIdx.x]);
        __syncthreads();
        for (uint32_t k = threadIdx.x; k < staged; k += kQCountThreads) {
            const uint32_t m = sm_side[k], b = (m - lo) >> bshift, at = sm_bbase[b] + sm_pos[k];
            if (at < kQBucketCap) list[b * kQBucketCap + at] = m;
        }
    } else {
        for (int k = threadIdx.x; k < kQSideBins; k += kQCountThreads) { const uint32_t c = sm_side[k]; if (c) atomicAdd(&hist_bracket[k], c); }
    }
    if (!last_cta_done(&ctl->ticket[1])) return;

    // ---- finish: everything the CTAs left is exact
    const unsigned long long nnz = __ldcg(&ctl->count_nz);
    if (nnz == 0) {
        if (threadIdx.x == 0) { out->value = 0.f; out->pad = 0; out->nnz = 0; }
        return;
    }
    unsigned long long r = (unsigned long long)ceil(q * (double)nnz);
    if (r < 1) r = 1;
    if (r > nnz) r = nnz;
    const unsigned long long below = nnz - __ldcg(&ctl->count_ge);
    constexpr int PER = kQSideBins / kQCountThreads;
    uint32_t bin;
    unsigned long long rib;
    if (DT == LGN_BF16) {
        unsigned long long inside;
        const unsigned long long mine = own_sum<PER, false>(hist_bracket);
        const unsigned long long before = cta_exclusive_scan(mine, sm, &inside);
        if (hi16 - lo16 > (uint32_t)kQSideBins || r <= below || r - below > inside) {
            if (threadIdx.x == 0) ctl->fallback = 1u;
            return;
        }
        locate<PER, false>(hist_bracket, r - below, mine, before, &bin, &rib);
        if (threadIdx.x == 0) { out->value = u2f((lo16 + bin) << 16); out->pad = 0; out->nnz = nnz; }
        return;
    }
    // which list holds rank r - below, and which rank in it
    __shared__ uint32_t sm_which, sm_length;
    __shared__ unsigned long long sm_k;
    unsigned long long listed;
    const unsigned long long mine = threadIdx.x < kQBuckets ? (unsigned long long)__ldcg(&ctl->bucket[threadIdx.x]) : 0ull;
    const unsigned long long before = cta_exclusive_scan(mine, sm, &listed);
    if (r <= below || r - below > listed) {
        if (threadIdx.x == 0) ctl->fallback = 1u;
        return;
    }
    if (r - below > before && r - below <= before + mine) { sm_which = threadIdx.x; sm_length = (uint32_t)mine; sm_k = r - below - before; }
    __syncthreads();
    const uint32_t which = sm_which, count = sm_length;
    if (count > kQBucketCap) {                              // that list is short of some of its patterns
        if (threadIdx.x == 0) ctl->fallback = 1u;
        return;
    }
    // radix selection on d = pattern - first (< 2^bshift), up to 12 bits a pass from the top
    unsigned long long k = sm_k;
    const uint32_t first = lo + (which << bshift);
    const uint4 *list4 = reinterpret_cast<const uint4 *>(list + (size_t)which * kQBucketCap);
    uint32_t prefix = 0u;
    for (int top = bshift; top > 0;) {
        const int shift = top > 12 ? top - 12 : 0;
        const uint32_t digit_mask = (1u << (top - shift)) - 1u;
        __syncthreads();
        for (int b = threadIdx.x; b < kQSideBins; b += kQCountThreads) sm_side[b] = 0u;
        __syncthreads();
        for (uint32_t i0 = 4u * threadIdx.x; i0 < count; i0 += 32u * kQCountThreads) {      // 8 x 16 bytes in flight per thread
            uint4 d[8];
            #pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t i = i0 + (uint32_t)j * 4u * kQCountThreads;
                d[j] = i < count ? __ldcg(list4 + i / 4u) : make_uint4(0u, 0u, 0u, 0u);
            }
            #pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t i = i0 + (uint32_t)j * 4u * kQCountThreads;
                const uint32_t e[4] = { d[j].x - first, d[j].y - first, d[j].z - first, d[j].w - first };
                #pragma unroll
                for (int t = 0; t < 4; ++t)                // the last 16 bytes may reach past the list's end
                    if (i + t < count && (e[t] >> top) == prefix) atomicAdd(&sm_side[(e[t] >> shift) & digit_mask], 1u);
            }
        }
        __syncthreads();
        unsigned long long total;
        const unsigned long long own = own_sum<PER, true>(sm_side);
        const unsigned long long ahead = cta_exclusive_scan(own, sm, &total);
        locate<PER, true>(sm_side, k, own, ahead, &bin, &rib);
        prefix = (prefix << (top - shift)) | bin;
        k = rib;
        top = shift;
    }
    if (threadIdx.x == 0) { out->value = u2f(first + prefix); out->pad = 0; out->nnz = nnz; }
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
    uint32_t *hist_low = hist_top + kQTopBins;              // also: the sample's histogram, then the bf16 bracket's bins
    uint32_t *list = hist_low + kQLowBins + kQTopBins + kQCoarse;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return LGN_ERR_CUDA;
    const size_t smem = sizeof(uint32_t) * (size_t)kQTopBins;
    const bool f32 = dt == LGN_F32;
    const void *top = f32 ? reinterpret_cast<const void *>(&quantile_top_kernel<LGN_F32>)
                          : reinterpret_cast<const void *>(&quantile_top_kernel<LGN_BF16>);
    const void *sample = f32 ? reinterpret_cast<const void *>(&quantile_sample_kernel<LGN_F32>)
                             : reinterpret_cast<const void *>(&quantile_sample_kernel<LGN_BF16>);
    if (cudaFuncSetAttribute(top, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncSetAttribute(sample, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return LGN_ERR_CUDA;
    if (cudaMemsetAsync(ws, 0, kQZeroedBytes, st) != cudaSuccess) return LGN_ERR_CUDA;
    const unsigned chunk = f32 ? 8u : 16u;
    const uint64_t nchunks = (n + chunk - 1) / chunk;
    auto grid_for = [&](uint64_t chunks, uint64_t per_cta, uint64_t most) {
        const uint64_t want = (chunks + per_cta - 1) / per_cta;
        return (unsigned)(want < 1 ? 1 : (want > most ? most : want));
    };
    const unsigned grid = grid_for(nchunks, (uint64_t)kQThreads * kQInFlight, (uint64_t)sms);
    // Sample size.  The bracket holds about 2 kQSigmas sqrt(q (1 - q) / m) of the nonzero elements (m = nonzero
    // elements of the sample).  fp32: m is chosen so that this is a quarter of the list for a tensor without
    // zeros; a sample of more than an eighth of the tensor is not worth its read.  bf16 brackets are a few
    // values wide whatever m is.
    uint64_t elems = kQSampleMin;
    if (f32) {
        const double root = 8.0 * kQSigmas * sqrt(q * (1.0 - q)) * (double)n / (double)kQListCap;
        if (root * root > (double)elems) elems = (uint64_t)(root * root);
    }
    const int direct = n < kQDirect || elems > n / 8;
    log_line("quantile: n=%llu %s q=%.17g -> %s", (unsigned long long)n, f32 ? "fp32" : "bf16", q,
             direct ? (n < kQDirect ? "radix selection (tensor below 2^24 elements)" : "radix selection (the sample would pass n / 8)")
                    : "one read around a bracket from a sample");
    if (!direct) log_line("quantile: sample of %llu elements", (unsigned long long)elems);
    bool first = true, ok = true;                            // the first kernel of the call follows the memset in plain stream order
    auto launch = [&](const void *fn, unsigned blocks, unsigned threads, size_t shared, void **args) {
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3(blocks); cfg.blockDim = dim3(threads); cfg.dynamicSmemBytes = shared; cfg.stream = st;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = first ? 0 : 1;
        first = false;
        if (cudaLaunchKernelExC(&cfg, fn, args) != cudaSuccess) ok = false;
    };
    uint32_t *hist_sample = hist_low + kQLowBins, *coarse = hist_sample + kQTopBins;
    int always = direct;
    if (!direct) {
        uint64_t nsample = elems / chunk;
        if (nsample > nchunks) nsample = nchunks;
        uint32_t nsample32 = (uint32_t)nsample, step = (uint32_t)(nchunks / nsample);
        const unsigned sgrid = grid_for(nsample, (uint64_t)kQThreads * 2, (uint64_t)sms);
        const unsigned cgrid = grid_for(nchunks, (uint64_t)kQCountThreads * kQInFlight * kQRoundSteps, (uint64_t)sms * 2);
        void *sargs[] = { &g, &n, &nsample32, &step, &hist_sample, &coarse, &q, &ctl };
        launch(sample, sgrid, kQThreads, smem, sargs);
        void *cargs[] = { &g, &n, &q, &ctl, &list, &hist_low, &out_dev };
        launch(f32 ? reinterpret_cast<const void *>(&quantile_count_kernel<LGN_F32>)
                   : reinterpret_cast<const void *>(&quantile_count_kernel<LGN_BF16>), cgrid, kQCountThreads, 0, cargs);
    }
    void *targs[] = { &g, &n, &hist_top, &q, &ctl, &out_dev, &always };
    launch(top, grid, kQThreads, smem, targs);
    if (f32) {
        void *largs[] = { &g, &n, &ctl, &hist_low, &out_dev };
        launch(reinterpret_cast<const void *>(&quantile_low_kernel), grid, kQThreads, 0, largs);
    }
    return ok && cudaGetLastError() == cudaSuccess ? LGN_OK : LGN_ERR_CUDA;
}
