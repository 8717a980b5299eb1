// Workspace layout, tile runners and kernel templates of the grouped path.  Included by the
// host side (lgn.cu) and by the translation units that instantiate the kernels
// (lgn_inst_*.cu): the instances are spread over several files so that they compile in
// parallel.
//
// One persistent kernel runs the whole path for a list of tensors.  Work is cut
// into tiles of kTileElems elements; tiles of all layers sit in one queue, in an
// order the host chooses, and CTAs pop them with one atomic each:
//
//   statistics tile : log2|g| partial sums of the tile -> its slot in the partial
//                     array; the CTA that completes a layer's last statistics tile
//                     adds the layer's partials in a fixed order, evaluates the
//                     closed form (Eq. 8 inverse or Eq. 4 argmin) in fp64 and
//                     publishes the result with a release store
//   apply tile      : waits (bounded) for that publication, then prunes (Eq. 5) or
//                     quantises and packs (Eq. 1-2) the tile
//
// A statistics tile never waits, and a layer's statistics tiles precede its apply
// tiles in the queue, so every wait is on work already handed to a running CTA.
#pragma once

#include <cstdio>
#include <cstring>

#include <cuda_runtime.h>

#include "lgn.h"
#include "lgn_closed_form.cuh"
#include "lgn_device.cuh"

namespace lgn {

// ------------------------------------------------------------------ workspace layout
struct WsHeader {
    uint32_t queue_head;
    uint32_t error;
    Weyl     weyl;                       // key-schedule increments, read as run-time values
    uint32_t pad[60];
};
static_assert(sizeof(WsHeader) == 256, "header is one 256-byte block");

constexpr int32_t kModeStatsOnly = 2;

struct alignas(16) LayerState {          // written by the set-up launch, then read-only
    const void         *g;
    void               *out;
    uint64_t            n;
    uint64_t            seed;
    double              S;
    double              mu_override, sigma_override;
    lgn_stats_t        *stats_out;       // may be null
    lgn_layer_result_t *result_out;      // may be null
    uint32_t            ntiles;
    uint32_t            partial0;        // first slot of this layer in the partial array
    int32_t             dt, mode, nbits, rounding, use_override, scale_mode;
    const uint8_t      *mask;            // right-mode mask of a bi-modal gradient, or null
    int32_t             counters;        // the apply tiles add their counts to result_out
    int32_t             pad;
};
static_assert(sizeof(LayerState) == 128, "LayerState layout");

// Layers that need the extended statistics tile (mask and / or max|g|); their
// statistics runs carry phase kPhaseStatsExt in the queue.
static inline bool needs_ext_stats(const LayerState &L) {
    return L.mask != nullptr || L.scale_mode == LGN_SCALE_FROM_MAX;
}
constexpr uint32_t kPhaseStats = 0, kPhaseApply = 1, kPhaseStatsExt = 2;

struct alignas(16) LayerDyn {            // zeroed by the set-up launch, written by the kernel
    uint32_t    done;                    // statistics tiles completed
    uint32_t    ready;                   // 1 once tau / q below are valid
    float       tau;
    int32_t     status;
    QuantParams q;
};
static_assert(sizeof(LayerDyn) == 80, "LayerDyn layout");

struct alignas(16) Segment {             // a run of consecutive queue items
    uint32_t first_item;
    uint32_t ntiles;
    uint32_t layer;
    uint32_t phase;                      // 0 statistics, 1 apply, 2 statistics with a mask and / or max|g|
    uint32_t tile_begin;                 // first tile of the layer this run covers
    uint32_t reverse;                    // walk the run from its last tile down
    uint32_t pad[2];
};
static_assert(sizeof(Segment) == 32, "Segment layout");

struct alignas(16) Partial {
    double             s1, s2;           // sums of log2|g| and its square over the tile's nonzeros
    unsigned long long cnt;
    uint32_t           right;            // extended tiles: entries of the right mode in the tile; else 0
    float              amax;             // extended tiles: largest magnitude in the tile; else 0
};
static_assert(sizeof(Partial) == 32, "Partial layout");

struct WsLayout {
    size_t states, dyn, segs, partials, total;
    uint32_t nseg_max;
    uint64_t total_tiles;
};

static inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Tiles of small calls.  A call of fewer tiles than the grid has CTAs cannot fill the GPU: each of its
// CTAs streams one 128 KiB tile alone, bound by the latency of its own loads; a call of little more than
// one round of the grid ends each pass with a second round that few CTAs run.  Such calls (fewer tiles than
// one and a half rounds) take tiles of a quarter of the bytes (a flat 2^20-element fp32 tensor: 128 CTAs of
// 32 KiB instead of 32 of 128 KiB).
// kSmallCallTiles bounds "small" for the workspace layout, which knows no device: below it the layout has
// room for the small tiles' partial sums, and the kernels are chosen by the actual grid, never above it.
constexpr int kSmallTileElemsF32 = kTileElems / 4, kSmallTileElemsBf16 = kTileElems / 2;
constexpr uint64_t kSmallCallTiles = 1024;

static bool ws_layout(const uint64_t *n_per_layer, int L, WsLayout &w) {
    if (L < 0) return false;
    uint64_t tiles = 0;
    for (int k = 0; k < L; ++k) {
        if (n_per_layer[k] > (1ull << 44)) return false;
        tiles += (n_per_layer[k] + kTileElems - 1) / kTileElems;
    }
    // Room for the partial sums of small tiles: a small call has at most four times its standard tiles,
    // so three times kSmallCallTiles more slots serve every small call; added to every layout, so that the
    // workspace of a list of layers is enough for any subset of it (the host-buffer form runs subsets).
    tiles += 3 * kSmallCallTiles;
    if (tiles >= (1ull << 31)) return false;
    w.total_tiles = tiles;
    w.nseg_max = 2u * (uint32_t)L + 2u;
    w.states = sizeof(WsHeader);
    w.dyn = w.states + round_up(sizeof(LayerState) * (size_t)L, 256);
    w.segs = w.dyn + round_up(sizeof(LayerDyn) * (size_t)L, 256);
    w.partials = w.segs + round_up(sizeof(Segment) * (size_t)w.nseg_max, 256);
    w.total = w.partials + round_up(sizeof(Partial) * (size_t)tiles, 256);
    return true;
}

// ------------------------------------------------------------------ set-up launch
// Host bytes travel to the device inside the kernel parameter block: no pinned
// staging buffer, no synchronous copy, ordered on the stream like any launch.
// Two sizes: an image of up to kBlobBytes goes in one small launch; a larger one
// (more than a dozen layers) in launches of kBigBlobBytes each, so that a call with
// a hundred layers still has a single set-up launch.
constexpr int kBlobBytes = 3840;
constexpr int kBigBlobBytes = 32512;
template <int BYTES> struct BlobT { uint4 v[BYTES / 16]; };

template <int BYTES>
__global__ void upload_kernel(const __grid_constant__ BlobT<BYTES> blob, uint4 *dst, int nvec) {
    // A compute kernel launched behind this one with programmatic stream
    // serialisation may be scheduled now; it waits (griddepcontrol.wait) for this
    // grid to finish and its stores to be visible before it reads the image.
    asm volatile("griddepcontrol.launch_dependents;");
    for (int i = threadIdx.x; i < nvec; i += blockDim.x) dst[i] = blob.v[i];
}

template <int BYTES>
static void upload_image(const unsigned char *image, size_t used, unsigned char *base, cudaStream_t stream) {
    for (size_t off = 0; off < used; off += BYTES) {
        BlobT<BYTES> blob;
        const size_t nb = used - off < (size_t)BYTES ? used - off : (size_t)BYTES;
        memcpy(blob.v, image + off, nb);                    // nb is a multiple of 16
        upload_kernel<BYTES><<<1, BYTES >= 8192 ? 256 : 128, 0, stream>>>(blob, reinterpret_cast<uint4 *>(base + off), (int)(nb / 16));
    }
}

static int upload_launches(size_t used) {
    return used <= (size_t)kBlobBytes ? 1 : (int)((used + kBigBlobBytes - 1) / kBigBlobBytes);
}

// The uploaded image is [header | states | dyn | segments]: it ends after the
// segment table (at most two runs per layer plus the terminator).
static size_t upload_bytes(const WsLayout &w, int L) {
    return w.segs + sizeof(Segment) * (2u * (size_t)L + 1u);
}

// ------------------------------------------------------------------ device helpers
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(uint32_t *p, uint32_t v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

// ------------------------------------------------------------------ tile runners
// Every pass has one hot body (whole tile inside the tensor; for quantisation
// also the fast code path, for pruning a normal-range threshold) that
// specialised kernels inline, and one general body (ragged last tile, any layer
// scale, any threshold) kept out of line so that it costs the hot path no
// registers.
// The out-of-line statistics tile: ragged last tiles, and the extended form (a
// right-mode mask and / or max|g|).  Does the whole item: the tile, the CTA
// reduction (one barrier) and the partial.
template <int DT, int TILE>
__device__ __noinline__ void run_stats_tile_slow(const LayerState &L, uint32_t tile, bool ext, Partial *partials, double *sm);

// One tile's sums: per-warp shuffle tree, eight warp results through shared
// memory, added in warp order by thread 0, which also stores the tile's partial.
// One barrier; `sm` is reused only after the caller's next barrier.
template <int DT, bool INLINE_HOT, int TILE>
__device__ __forceinline__ void run_stats_tile(const LayerState &L, uint32_t tile, bool ext, Partial *partials, double *sm) {
    const uint64_t base = (uint64_t)tile * TILE;
    if (!INLINE_HOT || ext || base + TILE > L.n) { run_stats_tile_slow<DT, TILE>(L, tile, ext, partials, sm); return; }
    StatsAcc acc;
    stats_tile<DT, true, TILE>(L.g, base, L.n, acc);
    #pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        acc.s1 += __shfl_down_sync(0xFFFFFFFFu, acc.s1, off);
        acc.s2 += __shfl_down_sync(0xFFFFFFFFu, acc.s2, off);
        acc.cnt += __shfl_down_sync(0xFFFFFFFFu, acc.cnt, off);
    }
    const int w = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) {
        sm[w] = acc.s1; sm[kWarps + w] = acc.s2; sm[2 * kWarps + w] = __longlong_as_double((long long)acc.cnt);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        Partial p;
        p.s1 = 0.0; p.s2 = 0.0; p.cnt = 0; p.right = 0u; p.amax = 0.f;
        #pragma unroll
        for (int k = 0; k < kWarps; ++k) {
            p.s1 += sm[k]; p.s2 += sm[kWarps + k];
            p.cnt += (unsigned long long)__double_as_longlong(sm[2 * kWarps + k]);
        }
        partials[L.partial0 + tile] = p;
    }
}

template <int DT, int TILE>
__device__ __noinline__ void run_stats_tile_slow(const LayerState &L, uint32_t tile, bool ext, Partial *partials, double *sm) {
    StatsAcc acc;
    const uint64_t base = (uint64_t)tile * TILE;
    if (!ext)        stats_tile<DT, false, TILE>(L.g, base, L.n, acc);
    else if (L.mask) stats_tile_ext<DT, true, TILE>(L.g, L.mask, base, L.n, acc);
    else             stats_tile_ext<DT, false, TILE>(L.g, nullptr, base, L.n, acc);
    warp_reduce(acc, 32);
    const int w = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) {
        sm[w] = acc.s1; sm[kWarps + w] = acc.s2; sm[2 * kWarps + w] = __longlong_as_double((long long)acc.cnt);
        sm[3 * kWarps + w] = __longlong_as_double((long long)acc.right); sm[4 * kWarps + w] = (double)acc.amax;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        Partial p;
        p.s1 = 0.0; p.s2 = 0.0; p.cnt = 0; p.right = 0u; p.amax = 0.f;
        #pragma unroll
        for (int k = 0; k < kWarps; ++k) {
            p.s1 += sm[k]; p.s2 += sm[kWarps + k];
            p.cnt += (unsigned long long)__double_as_longlong(sm[2 * kWarps + k]);
            p.right += (uint32_t)__double_as_longlong(sm[3 * kWarps + k]);
            p.amax = fmaxf(p.amax, (float)sm[4 * kWarps + k]);
        }
        partials[L.partial0 + tile] = p;
    }
}

// The general bodies always count (they are not the fast path); `tc` may be null.
template <int DT, int TILE>
__device__ __noinline__ void prune_tile_general(const void *g, void *out, uint64_t base, uint64_t n,
                                                float tau, uint64_t seed, const Weyl &wy, TileCounts *tc) {
    TileCounts local;
    prune_tile<DT, false, TILE, true>(g, out, base, n, tau, seed, wy, &local);
    if (tc) { tc->a += local.a; tc->b += local.b; }
}

// COUNT: the inlined hot body counts too (the instances that serve groups which ask for counters).
template <int DT, bool INLINE_HOT, int TILE, bool COUNT = false>
__device__ __forceinline__ void run_prune_tile(const void *g, void *out, uint64_t n, uint32_t tile,
                                               float tau, uint64_t seed, const Weyl &wy, TileCounts *tc = nullptr) {
    const uint64_t base = (uint64_t)tile * TILE;
    const bool tiny = tau > 0.f && tau < kPruneFastMin;       // alpha*2^-16 inexact, or alpha*eps could round to zero
    if (INLINE_HOT && base + TILE <= n && !tiny) prune_tile<DT, true, TILE, COUNT>(g, out, base, n, tau, seed, wy, tc);
    else                                         prune_tile_general<DT, TILE>(g, out, base, n, tau, seed, wy, tc);
}

template <int DT, int NBITS, bool SR, int TILE>
__device__ __noinline__ void quant_tile_general(const void *g, uint32_t *codes, uint64_t base, uint64_t n,
                                                uint64_t total_words, const QuantParams &q, uint64_t seed,
                                                const Weyl &wy, TileCounts *tc) {
    TileCounts local;
    quant_tile<DT, NBITS, SR, false, false, TILE, true>(g, codes, base, n, total_words, q, seed, wy, &local);
    if (tc) { tc->a += local.a; tc->b += local.b; }
}

template <int DT, int NBITS, bool SR, bool INLINE_HOT, int TILE, bool COUNT = false>
__device__ __forceinline__ void run_quant_tile(const void *g, void *out, uint64_t n, uint32_t tile,
                                               const QuantParams &q, uint64_t seed, const Weyl &wy, TileCounts *tc = nullptr) {
    const uint64_t base = (uint64_t)tile * TILE;
    const uint64_t total_words = (n * (uint64_t)NBITS + 31) >> 5;
    uint32_t *codes = static_cast<uint32_t *>(out);
    if (INLINE_HOT && base + TILE <= n && q.K >= 1 && q.K <= 255)
        quant_tile<DT, NBITS, SR, true, true, TILE, COUNT>(g, codes, base, n, total_words, q, seed, wy, tc);
    else
        quant_tile_general<DT, NBITS, SR, TILE>(g, codes, base, n, total_words, q, seed, wy, tc);
}

// Adds a tile's counts to its layer's result record: one warp-wide sum and, from lane 0, one
// atomic per field.  finalize_layer has stored the record, with the counters at their starting
// values (see there), before any apply tile of the layer can run.
__device__ __forceinline__ void flush_counts(const LayerState &L, const TileCounts &tc) {
    if (!L.counters || L.result_out == nullptr) return;
    const unsigned long long a = __reduce_add_sync(0xFFFFFFFFu, tc.a), b = __reduce_add_sync(0xFFFFFFFFu, tc.b);
    if ((threadIdx.x & 31) != 0) return;
    lgn_layer_result_t *r = L.result_out;
    if (L.mode == LGN_MODE_PRUNE) {
        atomicAdd(reinterpret_cast<unsigned long long *>(&r->n_zero_out), 0ull - a);    // starts at n
        atomicAdd(reinterpret_cast<unsigned long long *>(&r->n_snapped), a - b);        // kept but not above alpha
    } else {
        atomicAdd(reinterpret_cast<unsigned long long *>(&r->n_zero_out), 0ull - a);    // starts at n
        atomicAdd(reinterpret_cast<unsigned long long *>(&r->n_underflow), 0ull - a);   // starts at nnz
        atomicAdd(reinterpret_cast<unsigned long long *>(&r->n_saturated), b);
    }
}

// run-time dispatch for groups whose layers differ in type, mode or width
template <int DT>
__device__ __forceinline__ void run_quant_tile_any(const void *g, void *out, uint64_t n, uint32_t tile, int nbits,
                                                   const QuantParams &q, bool sr, uint64_t seed, const Weyl &wy,
                                                   TileCounts *tc) {
    #define LGN_Q(NB) \
        if (sr) run_quant_tile<DT, NB, true, false, kTileElems>(g, out, n, tile, q, seed, wy, tc); \
        else    run_quant_tile<DT, NB, false, false, kTileElems>(g, out, n, tile, q, seed, wy, tc);
    switch (nbits) {
        case 4: LGN_Q(4) break;
        case 5: LGN_Q(5) break;
        case 6: LGN_Q(6) break;
        case 7: LGN_Q(7) break;
        default: LGN_Q(8) break;
    }
    #undef LGN_Q
}

// floor(log2 a) of a positive finite fp32 value, from its pattern (subnormals included).
__host__ __device__ inline int floor_log2_f32(float a) {
    uint32_t b;
    memcpy(&b, &a, 4);
    b &= 0x7FFFFFFFu;
    const int e = (int)(b >> 23);
    if (e) return e - 127;
    int top = -1;
    for (int k = 22; k >= 0; --k) if ((b >> k) & 1u) { top = k; break; }
    return top - 149;
}

// choose_format with the candidate splits spread over the lanes of a warp (lane k evaluates Eq. 4
// for n2 = k + 1): the same arithmetic per candidate and the same choice (the smallest n2 among
// the minima) as the sequential form, in the time of one evaluation instead of nbits - 1.
// All 32 lanes call.
__device__ __forceinline__ void choose_format_warp(double mu, double sigma, int nbits, lgn_fp_format_t &f) {
    const double s = clamp_sigma(sigma);
    int n2 = (int)(threadIdx.x & 31) + 1;
    double eta = n2 <= nbits - 1 ? expected_rel_err(s, nbits - 1 - n2, n2) : __longlong_as_double(0x7FF0000000000000ll);
    #pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const double oe = __shfl_down_sync(0xFFFFFFFFu, eta, off);
        const int on = __shfl_down_sync(0xFFFFFFFFu, n2, off);
        if (oe < eta || (oe == eta && on < n2)) { eta = oe; n2 = on; }
    }
    n2 = __shfl_sync(0xFFFFFFFFu, n2, 0);
    f.nbits = nbits;
    f.exp_bits = n2;
    f.man_bits = nbits - 1 - n2;
    f.scale_exp = (int32_t)floor(mu / kLn2 + 0.5);
}

// Adds up a layer's partials (thread t takes slots t, t+kThreads, ... in order,
// then the fixed tree), turns them into mu, sigma, and evaluates the closed form (on warp 0:
// every lane carries the same values, lane 0 stores them).
static __device__ __noinline__ void finalize_layer(const LayerState &L, LayerDyn *D, const Partial *partials, double *sm) {
    StatsAcc acc;
    for (uint32_t t = threadIdx.x; t < L.ntiles; t += kThreads) {
        const Partial *p = partials + L.partial0 + t;
        acc.s1 += __ldcg(&p->s1);
        acc.s2 += __ldcg(&p->s2);
        acc.cnt += __ldcg(&p->cnt);
        acc.right += __ldcg(&p->right);
        acc.amax = fmaxf(acc.amax, __ldcg(&p->amax));
    }
    block_reduce(acc, sm);
    if (threadIdx.x >= 32) return;
    acc.s1 = __shfl_sync(0xFFFFFFFFu, acc.s1, 0);
    acc.s2 = __shfl_sync(0xFFFFFFFFu, acc.s2, 0);
    acc.cnt = __shfl_sync(0xFFFFFFFFu, acc.cnt, 0);
    acc.right = __shfl_sync(0xFFFFFFFFu, acc.right, 0);
    acc.amax = __shfl_sync(0xFFFFFFFFu, acc.amax, 0);
    const bool lead = threadIdx.x == 0;

    lgn_stats_t st;
    st.n = L.n;
    st.nnz = acc.cnt;
    st.sum_ln = st.sum_ln2 = st.mu = st.sigma = 0.0;
    if (acc.cnt) {
        const double inv = 1.0 / (double)acc.cnt;
        const double m2 = acc.s1 * inv;                       // mean of log2|g|
        double var = acc.s2 * inv - m2 * m2;
        if (!(var > 0.0)) var = 0.0;
        st.mu = m2 * kLn2;
        st.sigma = sqrt(var) * kLn2;
        st.sum_ln = acc.s1 * kLn2;
        st.sum_ln2 = acc.s2 * kLn2 * kLn2;
    }
    if (lead && L.stats_out) *L.stats_out = st;

    const double mu = L.use_override ? L.mu_override : st.mu;
    const double sigma = L.use_override ? L.sigma_override : st.sigma;
    double tau_used = 0.0;
    lgn_fp_format_t fmt;
    fmt.nbits = fmt.exp_bits = fmt.man_bits = fmt.scale_exp = 0;
    if (L.mode == LGN_MODE_PRUNE) {
        // l: the exact zeros, or with a mask the left mode (appendix, bi-modal pruning, step 1)
        const double zero_frac = 1.0 - (double)(L.mask ? acc.right : st.nnz) / (double)st.n;
        const double tau = acc.cnt ? threshold_for(mu, sigma, zero_frac, L.S) : 0.0;
        const float t = (L.dt == LGN_BF16) ? snap_threshold_bf16(tau) : snap_threshold_f32(tau);
        if (lead) D->tau = t;
        tau_used = (double)t;
    } else if (L.mode == LGN_MODE_QUANTIZE) {
        if (acc.cnt) {
            choose_format_warp(mu, sigma, L.nbits, fmt);
            if (L.scale_mode == LGN_SCALE_FROM_MAX)               // Algorithm 1: the maximum in the top binade
                fmt.scale_exp = floor_log2_f32(acc.amax) - ((1 << (fmt.exp_bits - 1)) - 1);
        } else {                                              // all zero: every code is 0 anyway
            fmt.nbits = L.nbits; fmt.exp_bits = 1; fmt.man_bits = L.nbits - 2; fmt.scale_exp = 0;
        }
        if (lead) D->q = make_quant_params(fmt);
    }
    if (!lead) return;
    if (L.result_out) {
        lgn_layer_result_t r;
        r.stats = st; r.tau = tau_used; r.fmt = fmt; r.status = LGN_OK;
        r.max_abs = acc.amax; r.n_right_mode = L.mask ? acc.right : 0ull;
        // Counters start where the apply tiles' atomics (flush_counts) leave the final values:
        // zeros out = n - nonzero outputs; underflows = nnz - nonzero codes (a nonzero code
        // always comes from a nonzero input).
        r.n_zero_out = L.counters ? st.n : 0ull;
        r.n_underflow = (L.counters && L.mode == LGN_MODE_QUANTIZE) ? st.nnz : 0ull;
        r.n_snapped = 0ull; r.n_saturated = 0ull;
        *L.result_out = r;
    }
    __threadfence();
    // A waiter that gave up on this layer before now has skipped tiles: its verdict
    // stands, whichever of the two stores to the record's status lands first.
    if (atomicAdd(&D->status, 0) != 0 && L.result_out) {
        *(volatile int32_t *)&L.result_out->status = LGN_ERR_TIMEOUT;
        __threadfence();
    }
    st_release(&D->ready, 1u);
}

__device__ __forceinline__ QuantParams load_quant_params(const LayerDyn *D) {
    const uint4 *src = reinterpret_cast<const uint4 *>(&D->q);   // written by another CTA: read through L2
    const uint4 a = __ldcg(src), b = __ldcg(src + 1), c = __ldcg(src + 2), d = __ldcg(src + 3);
    const uint32_t raw[16] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w, c.x, c.y, c.z, c.w, d.x, d.y, d.z, d.w};
    QuantParams q;
    memcpy(&q, raw, sizeof q);
    return q;
}

// ------------------------------------------------------------------ the persistent kernel
constexpr uint32_t kMaxPolls = 1u << 19;      // x ~1 us per poll (acquire load + back-off): about half a second
constexpr int kAny = -1;                      // template value: decided per layer at run time

// DT, MODE, NBITS, SR fix what every layer of the group has in common, so that
// the hot tile bodies are inlined and nothing else is compiled into the kernel;
// kAny for all four is the general kernel for mixed groups.  EXT: the group's
// layers may ask for the extended statistics tile (a right-mode mask, max|g|);
// every specialised kernel exists without and (as a second instance) with it, so a
// group that does not ask pays nothing for it.
// Resident CTAs per SM the grouped kernel is compiled for: three (80 registers, no spills), which
// measured 2-4 % faster than four (64 registers, some spills) on every fp32 workload and on bf16
// with 32768-element tiles; the bf16 instances with 65536-element tiles keep four (ResNet-50 bf16
// pruning: -1.6 % at three); two is slower everywhere.
template <int DT, int TILE>
constexpr int compress_min_ctas() { return (DT == LGN_BF16 && TILE > kTileElems) ? kMinCtas : kMinCtas - 1; }

template <int DT, int MODE, int NBITS, int SR, bool EXT = false, int TILE = kTileElems>
__global__ void __launch_bounds__(kThreads, compress_min_ctas<DT, TILE>())
compress_kernel(WsHeader *hdr, const LayerState *states, LayerDyn *dyn, const Segment *segs,
                int num_layers, uint32_t total_items, Partial *partials) {
    __shared__ double sm_red[5 * kWarps];
    __shared__ uint32_t sm_item[2];
    __shared__ uint32_t sm_fin[2];               // layer + 1 whose statistics this CTA has just completed
    __shared__ uint32_t sm_flag;
    constexpr bool kSpecial = DT != kAny;

    // Launched with programmatic stream serialisation behind the last set-up
    // launch: the CTAs may already be resident while that launch runs, and wait
    // here until it has finished and the workspace image is visible.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (blockIdx.x == 0) {                       // layers with no elements have no tiles: answer here
        for (int k = threadIdx.x; k < num_layers; k += kThreads) {
            const LayerState &L = states[k];
            if (L.ntiles != 0) continue;
            lgn_stats_t st;
            st.n = 0; st.nnz = 0; st.sum_ln = st.sum_ln2 = st.mu = st.sigma = 0.0;
            if (L.stats_out) *L.stats_out = st;
            if (L.result_out) {
                lgn_layer_result_t r;
                memset(&r, 0, sizeof r);
                r.stats = st;
                if (L.mode == LGN_MODE_QUANTIZE) { r.fmt.nbits = L.nbits; r.fmt.exp_bits = 1; r.fmt.man_bits = L.nbits - 2; }
                *L.result_out = r;
            }
        }
    }
    Weyl wy;
    wy.w0 = __ldcg(&hdr->weyl.w0);
    wy.w1 = __ldcg(&hdr->weyl.w1);

    // Thread 0 keeps one queue item in hand: the next pop is issued as soon as
    // the current item is known, so its latency hides behind the tile's work.
    uint32_t next_item = 0, fin_layer1 = 0;      // thread 0 only
    if (threadIdx.x == 0) next_item = atomicAdd(&hdr->queue_head, 1u);
    uint32_t seg = 0;
    int ready_layer = -1;                        // layer whose closed form this CTA has already seen published
    for (uint32_t it = 0;; ++it) {
        if (threadIdx.x == 0) { sm_item[it & 1] = next_item; sm_fin[it & 1] = fin_layer1; fin_layer1 = 0; }
        __syncthreads();
        const uint32_t item = sm_item[it & 1];
        const uint32_t fin = sm_fin[it & 1];
        if (threadIdx.x == 0 && item < total_items) next_item = atomicAdd(&hdr->queue_head, 1u);
        if (fin) {                               // this CTA stored the last partial of layer fin-1
            __threadfence();
            finalize_layer(states[fin - 1], dyn + (fin - 1), partials, sm_red);
        }
        if (item >= total_items) break;
        while (item >= segs[seg].first_item + segs[seg].ntiles) ++seg;
        const Segment sg = segs[seg];
        uint32_t t = item - sg.first_item;
        if (sg.reverse) t = sg.ntiles - 1u - t;
        const uint32_t tile = sg.tile_begin + t;
        const LayerState &L = states[sg.layer];
        LayerDyn *D = dyn + sg.layer;

        if (sg.phase != kPhaseApply) {
            const bool ext = (EXT || !kSpecial) && sg.phase == kPhaseStatsExt;
            if constexpr (kSpecial) {
                run_stats_tile<DT, true, TILE>(L, tile, ext, partials, sm_red);
            } else {
                if (L.dt == LGN_BF16) run_stats_tile<LGN_BF16, false, kTileElems>(L, tile, ext, partials, sm_red);
                else                  run_stats_tile<LGN_F32, false, kTileElems>(L, tile, ext, partials, sm_red);
            }
            if (threadIdx.x == 0) {
                __threadfence();                                   // the partial before the ticket
                const uint32_t ticket = atomicAdd(&D->done, 1u);
                if (ticket == L.ntiles - 1u) fin_layer1 = sg.layer + 1u;   // acted on at the next barrier
            }
        } else {
            if ((int)sg.layer != ready_layer) {
                if (threadIdx.x == 0) {
                    // The wait is this layer's own: it ends early only when another waiter of
                    // the SAME layer has already given up.  Layers whose statistics are merely
                    // still running keep their full count whatever happened elsewhere.
                    // The count starts again whenever the queue has moved: the statistics tile
                    // this wait depends on may be in the hands of a CTA that is itself sitting
                    // out the wait of a layer that will never complete, and resumes after it.
                    // Such a CTA holds items that lie LATER in the queue than the one it waits
                    // for, so patience grows with the layer's position: the waiters of an
                    // earlier layer always give up, and move on, first.
                    const uint32_t limit = kMaxPolls * (1u + (sg.layer < 15u ? sg.layer : 15u));
                    uint32_t polls = 0, ok = 1, seen = *(volatile uint32_t *)&hdr->queue_head;
                    while (ld_acquire(&D->ready) == 0u) {
                        if (++polls > limit || *(volatile int32_t *)&D->status != 0) { ok = 0; break; }
                        if ((polls & 1023u) == 0u) {
                            const uint32_t head = *(volatile uint32_t *)&hdr->queue_head;
                            if (head != seen) { seen = head; polls = 0u; }
                        }
                        __nanosleep(100);
                    }
                    if (!ok) {
                        if (atomicCAS(&D->status, 0, (int32_t)LGN_ERR_TIMEOUT) == 0) atomicExch(&hdr->error, 1u);
                        __threadfence();                           // after a record finalize_layer may have stored
                        if (L.result_out) *(volatile int32_t *)&L.result_out->status = LGN_ERR_TIMEOUT;
                    }
                    sm_flag = ok;
                }
                __syncthreads();
                if (!sm_flag) continue;                            // timed out: skip the tile, keep draining
                ready_layer = (int)sg.layer;
            }
            // The instances with extended statistics also take the counters of the result record
            // (EXT is "everything beyond the plain path"); so does the general kernel.
            TileCounts tc;
            if constexpr (kSpecial && MODE == LGN_MODE_PRUNE) {
                const float tau = __ldcg(&D->tau);
                if (EXT && L.counters) run_prune_tile<DT, true, TILE, EXT>(L.g, L.out, L.n, tile, tau, L.seed, wy, &tc);
                else                   run_prune_tile<DT, true, TILE, false>(L.g, L.out, L.n, tile, tau, L.seed, wy, nullptr);
            } else if constexpr (kSpecial && MODE == LGN_MODE_QUANTIZE) {
                const QuantParams q = load_quant_params(D);
                if (EXT && L.counters) run_quant_tile<DT, NBITS, SR != 0, true, TILE, EXT>(L.g, L.out, L.n, tile, q, L.seed, wy, &tc);
                else                   run_quant_tile<DT, NBITS, SR != 0, true, TILE, false>(L.g, L.out, L.n, tile, q, L.seed, wy, nullptr);
            } else if constexpr (!kSpecial) {
                if (L.mode == LGN_MODE_PRUNE) {
                    const float tau = __ldcg(&D->tau);
                    if (L.dt == LGN_BF16) run_prune_tile<LGN_BF16, false, kTileElems>(L.g, L.out, L.n, tile, tau, L.seed, wy, &tc);
                    else                  run_prune_tile<LGN_F32, false, kTileElems>(L.g, L.out, L.n, tile, tau, L.seed, wy, &tc);
                } else {
                    const QuantParams q = load_quant_params(D);
                    const bool sr = L.rounding == LGN_ROUND_STOCHASTIC;
                    if (L.dt == LGN_BF16) run_quant_tile_any<LGN_BF16>(L.g, L.out, L.n, tile, L.nbits, q, sr, L.seed, wy, &tc);
                    else                  run_quant_tile_any<LGN_F32>(L.g, L.out, L.n, tile, L.nbits, q, sr, L.seed, wy, &tc);
                }
            }
            if constexpr (EXT || !kSpecial) flush_counts(L, tc);
        }
    }
}

// ------------------------------------------------------------------ stand-alone apply kernels
template <int DT>
__global__ void __launch_bounds__(kThreads, kMinCtas)
prune_kernel(const void *g, void *out, uint64_t n, uint32_t ntiles, float tau, uint64_t seed, Weyl wy) {
    for (uint32_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x)
        run_prune_tile<DT, true, kTileElems>(g, out, n, tile, tau, seed, wy);
}

template <int DT, int NBITS, int SR>
__global__ void __launch_bounds__(kThreads, kMinCtas)
quantize_kernel(const void *g, void *out, uint64_t n, uint32_t ntiles, const __grid_constant__ QuantParams q,
                uint64_t seed, Weyl wy) {
    for (uint32_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x)
        run_quant_tile<DT, NBITS, SR != 0, true, kTileElems>(g, out, n, tile, q, seed, wy);
}

// ------------------------------------------------------------------ kernel tables
// variant index: 0 statistics only, 1 prune, 2 + 2*(nbits-4) + sr quantise; with extended
// statistics: 12 prune, 13 + 2*(nbits-4) + sr quantise.  The tables are defined in lgn_inst_*.cu.
constexpr int kVariants = 23;
constexpr int kVariantPruneExt = 12, kVariantQuantExt0 = 13;
constexpr int kBigTileElems = 2 * kTileElems;        // bf16 tiles of large calls: 128 KiB of input, as for fp32
extern const void *const kCompressTableF32[kVariants];
extern const void *const kCompressTableBf16[kVariants];
extern const void *const kCompressTableBf16Big[kVariants];
extern const void *const kCompressTableF32Small[kVariants];
extern const void *const kCompressTableBf16Small[kVariants];
extern const void *const kCompressGeneral;
extern const void *const kQuantizeTable[2][10];
extern const void *const kPruneTable[2];

#define LGN_CK(DT, MODE, NB, SR, EXT, TILE) reinterpret_cast<const void *>(&compress_kernel<DT, MODE, NB, SR, EXT, TILE>)
#define LGN_CK_QUANT(DT, EXT, TILE) \
    LGN_CK(DT, LGN_MODE_QUANTIZE, 4, 0, EXT, TILE), LGN_CK(DT, LGN_MODE_QUANTIZE, 4, 1, EXT, TILE), \
    LGN_CK(DT, LGN_MODE_QUANTIZE, 5, 0, EXT, TILE), LGN_CK(DT, LGN_MODE_QUANTIZE, 5, 1, EXT, TILE), \
    LGN_CK(DT, LGN_MODE_QUANTIZE, 6, 0, EXT, TILE), LGN_CK(DT, LGN_MODE_QUANTIZE, 6, 1, EXT, TILE), \
    LGN_CK(DT, LGN_MODE_QUANTIZE, 7, 0, EXT, TILE), LGN_CK(DT, LGN_MODE_QUANTIZE, 7, 1, EXT, TILE), \
    LGN_CK(DT, LGN_MODE_QUANTIZE, 8, 0, EXT, TILE), LGN_CK(DT, LGN_MODE_QUANTIZE, 8, 1, EXT, TILE)
// one table row: every specialised kernel of a type and tile size, without and with extended statistics
#define LGN_CK_ROW(DT, TILE) { \
    LGN_CK(DT, kModeStatsOnly, kAny, kAny, false, TILE), LGN_CK(DT, LGN_MODE_PRUNE, kAny, kAny, false, TILE), \
    LGN_CK_QUANT(DT, false, TILE), LGN_CK(DT, LGN_MODE_PRUNE, kAny, kAny, true, TILE), LGN_CK_QUANT(DT, true, TILE) }

}  // namespace lgn
