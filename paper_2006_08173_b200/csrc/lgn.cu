// Host side and C entry points of the lognormal gradient-compression library: argument
// checks, the queue order, the set-up image and the launches.  The kernels themselves are in
// lgn_kernels.cuh, instantiated in lgn_inst_*.cu.
#include <cstdio>
#include <cstring>
#include <mutex>
#include <vector>

#include <cuda_runtime.h>

#include "lgn.h"
#include "lgn_log.h"
#include "lgn_kernels.cuh"

namespace lgn {

static int variant_of(int mode, int nbits, int rounding) {
    if (mode == kModeStatsOnly) return 0;
    if (mode == LGN_MODE_PRUNE) return 1;
    return 2 + 2 * (nbits - 4) + (rounding == LGN_ROUND_STOCHASTIC ? 1 : 0);
}

static const void *const *compress_table(int dt) { return dt == LGN_BF16 ? kCompressTableBf16 : kCompressTableF32; }

// ------------------------------------------------------------------ host side
static bool aligned8(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 7u) == 0; }
static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static bool aligned32(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }

// Resident CTAs of `fn` per SM x SM count of the current device: the size of a
// persistent grid.  A property of the device and the binary.
static int persistent_ctas(const void *fn) {
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kThreads, 0) != cudaSuccess) return -1;
    if (per_sm < 1) per_sm = 1;
    return sms * per_sm;
}

struct InternalLayer {
    lgn_layer_t          d;
    lgn_stats_t         *stats_out;
    lgn_layer_result_t  *result_out;
};

static lgn_status check_layer(const lgn_layer_t &d) {
    if (d.n > 0 && (d.g == nullptr || !aligned32(d.g))) return LGN_ERR_INVALID_ARG;
    if (d.dt != LGN_F32 && d.dt != LGN_BF16) return LGN_ERR_INVALID_ARG;
    if (d.mode == LGN_MODE_PRUNE) {
        if (!(d.S >= 0.0 && d.S < 1.0)) return LGN_ERR_INVALID_ARG;
    } else if (d.mode == LGN_MODE_QUANTIZE) {
        if (d.nbits < 4 || d.nbits > 8) return LGN_ERR_UNSUPPORTED;
        if (d.rounding != LGN_ROUND_NEAREST && d.rounding != LGN_ROUND_STOCHASTIC) return LGN_ERR_INVALID_ARG;
    } else if (d.mode != kModeStatsOnly) {
        return LGN_ERR_INVALID_ARG;
    }
    if (d.mode != kModeStatsOnly && d.n > 0) {
        if (d.out == nullptr || !(d.mode == LGN_MODE_PRUNE ? aligned32(d.out) : aligned16(d.out)))
            return LGN_ERR_INVALID_ARG;
        const size_t in_bytes = d.n * (d.dt == LGN_BF16 ? 2u : 4u);
        const size_t out_bytes = d.mode == LGN_MODE_PRUNE ? in_bytes : lgn_codes_bytes(d.n, d.nbits);
        const char *a = static_cast<const char *>(d.g), *b = static_cast<const char *>(d.out);
        if (a < b + out_bytes && b < a + in_bytes) return LGN_ERR_INVALID_ARG;    // overlap
    }
    if (d.mode == LGN_MODE_QUANTIZE) {
        if (d.scale_mode != LGN_SCALE_CENTRED && d.scale_mode != LGN_SCALE_FROM_MAX) return LGN_ERR_INVALID_ARG;
        if (d.right_mode != nullptr) return LGN_ERR_INVALID_ARG;       // the mask belongs to bi-modal pruning
    } else {
        if (d.scale_mode != 0) return LGN_ERR_INVALID_ARG;
        if (d.right_mode != nullptr && d.mode != LGN_MODE_PRUNE) return LGN_ERR_INVALID_ARG;
    }
    if (d.right_mode != nullptr && d.n > 0) {
        if (!aligned16(d.right_mode)) return LGN_ERR_INVALID_ARG;
        const char *m = static_cast<const char *>(d.right_mode), *b = static_cast<const char *>(d.out);
        const size_t out_bytes = d.n * (d.dt == LGN_BF16 ? 2u : 4u);
        if (m < b + out_bytes && b < m + d.n) return LGN_ERR_INVALID_ARG;   // the output would overwrite the mask
    }
    if (d.reserved != 0) return LGN_ERR_INVALID_ARG;
    if (d.use_override && !(d.sigma_override >= 0.0 && std::isfinite(d.mu_override) && std::isfinite(d.sigma_override)))
        return LGN_ERR_INVALID_ARG;
    return LGN_OK;
}

// Queue order.  A layer's apply tiles can start only once its statistics are
// complete (its last statistics tile may sit with a slow CTA) and its closed form
// (some microseconds on one warp) is published, so other work is placed between the
// two: statistics runs of the following layers are pulled forward until at least
// kLookaheadBytes of input lie between the end of S(k) and the start of A(k) (one
// following layer always).  The distance is worth far more than keeping a small
// layer in L2 for its second read: on the ResNet workloads 1 GiB measured 4 % (fp32
// pruning) to 10 % (FP6, bf16 pruning) faster than 96 MiB, with the gain levelling
// off from 512 MiB on; a call of less than 1 GiB simply takes all its statistics
// first.  A layer's apply run walks its tiles from the last one read back to the
// first, the order in which L2 may still hold the tail of a single tensor.
constexpr uint64_t kLookaheadBytes = 1024ull << 20;

static void build_queue(const std::vector<LayerState> &st, std::vector<Segment> &segs, uint32_t &total_items,
                        bool withhold_tile) {
    uint32_t item = 0;
    uint64_t bytes = 0;                                    // input bytes of all runs emitted so far
    auto push = [&](uint32_t layer, uint32_t phase) {
        if (st[layer].ntiles == 0) return;
        if (phase == 1 && st[layer].mode == kModeStatsOnly) return;
        Segment s;
        memset(&s, 0, sizeof s);
        s.first_item = item; s.ntiles = st[layer].ntiles; s.layer = layer;
        s.phase = phase == 1 ? kPhaseApply : (needs_ext_stats(st[layer]) ? kPhaseStatsExt : kPhaseStats);
        s.tile_begin = 0; s.reverse = phase;
        if (withhold_tile && layer == 0 && phase == 0) {   // self-test: layer 0 can never complete
            s.ntiles -= 1;
            if (s.ntiles == 0) return;
        }
        segs.push_back(s);
        item += s.ntiles;
        bytes += st[layer].n * (st[layer].dt == LGN_BF16 ? 2u : 4u);
    };
    const uint32_t L = (uint32_t)st.size();
    std::vector<uint64_t> bytes_after_stats(L, 0);
    uint32_t next_s = 0;
    for (uint32_t k = 0; k < L; ++k) {
        while (next_s < L && (next_s <= k + 1 || bytes - bytes_after_stats[k] < kLookaheadBytes)) {
            push(next_s, 0);
            bytes_after_stats[next_s] = bytes;
            ++next_s;
        }
        push(k, 1);
    }
    total_items = item;
}

static lgn_status run_layers(const std::vector<InternalLayer> &layers, void *ws, size_t ws_bytes, cudaStream_t stream,
                             bool withhold_tile = false) {
    const int L = (int)layers.size();
    if (L == 0) return LGN_OK;
    std::vector<uint64_t> ns(L);
    for (int k = 0; k < L; ++k) {
        lgn_status s = check_layer(layers[k].d);
        if (s != LGN_OK) {
            log_line("layer %d of %d refused: %s (n=%llu dt=%d mode=%d nbits=%d S=%g)", k, L, lgn_status_string(s),
                     (unsigned long long)layers[k].d.n, (int)layers[k].d.dt, (int)layers[k].d.mode, (int)layers[k].d.nbits, layers[k].d.S);
            return s;
        }
        ns[k] = layers[k].d.n;
    }
    WsLayout w;
    if (!ws_layout(ns.data(), L, w)) return LGN_ERR_UNSUPPORTED;
    if (ws == nullptr || !aligned16(ws)) return LGN_ERR_INVALID_ARG;
    if (ws_bytes < w.total) {
        log_line("workspace of %zu bytes refused: %d layers need %zu", ws_bytes, L, (size_t)w.total);
        return LGN_ERR_WORKSPACE;
    }

    std::vector<LayerState> st(L);
    for (int k = 0; k < L; ++k) {
        const lgn_layer_t &d = layers[k].d;
        LayerState &s = st[k];
        memset(&s, 0, sizeof s);
        s.g = d.g; s.out = d.out; s.n = d.n; s.seed = d.seed; s.S = d.S;
        s.mu_override = d.mu_override; s.sigma_override = d.sigma_override;
        s.stats_out = layers[k].stats_out; s.result_out = layers[k].result_out;
        s.dt = d.dt; s.mode = d.mode; s.nbits = d.nbits; s.rounding = d.rounding;
        s.use_override = d.use_override ? 1 : 0;
        s.scale_mode = d.scale_mode;
        s.mask = static_cast<const uint8_t *>(d.right_mode);
        s.counters = d.counters ? 1 : 0;
    }

    // one kernel per (type, mode, width, rounding) shared by all layers; the general one otherwise.
    // Extended statistics: the specialised kernels' second instances; mixed groups go general.
    bool any_ext = false, any_count = false, same = true;
    for (int k = 0; k < L; ++k) {
        any_count = any_count || st[k].counters;
        any_ext = any_ext || needs_ext_stats(st[k]) || st[k].counters;
        same = same && st[k].dt == st[0].dt && variant_of(st[k].mode, st[k].nbits, st[k].rounding) ==
                                                   variant_of(st[0].mode, st[0].nbits, st[0].rounding);
    }
    const void *fn = kCompressGeneral;
    if (same && !any_ext) fn = compress_table(st[0].dt)[variant_of(st[0].mode, st[0].nbits, st[0].rounding)];
    else if (same && st[0].mode == LGN_MODE_PRUNE) fn = compress_table(st[0].dt)[kVariantPruneExt];
    else if (same && st[0].mode == LGN_MODE_QUANTIZE)
        fn = compress_table(st[0].dt)[kVariantQuantExt0 + variant_of(st[0].mode, st[0].nbits, st[0].rounding) - 2];
    if (any_count || !same)                      // one layer asking, or the general kernel: every layer is counted
        for (int k = 0; k < L; ++k) st[k].counters = 1;
    int grid = persistent_ctas(fn);
    if (grid < 1) return LGN_ERR_CUDA;

    // Tile size.  128 KiB of input per tile is the measured optimum for both types: 32768 fp32
    // or 65536 bf16 elements.  The larger bf16 tile is used only when the call has enough of
    // them (eight rounds of the grid) for the coarser tail of the queue not to matter.
    uint32_t tile_elems = kTileElems;
    if (fn != kCompressGeneral && st[0].dt == LGN_BF16 && !withhold_tile) {
        uint64_t big_tiles = 0;
        for (int k = 0; k < L; ++k) big_tiles += st[k].n / kBigTileElems;
        if (big_tiles >= 8ull * (uint64_t)grid) {
            for (int v = 0; v < kVariants; ++v)
                if (kCompressTableBf16[v] == fn) { fn = kCompressTableBf16Big[v]; tile_elems = kBigTileElems; break; }
            grid = persistent_ctas(fn);
            if (grid < 1) return LGN_ERR_CUDA;
        }
    }
    // Small calls (fewer standard tiles than one and a half rounds of the grid; see kSmallCallTiles): smaller
    // tiles.  Measured on flat tensors: 2^24 elements (512 standard tiles for 444 CTAs, a second round that a
    // seventh of the CTAs run alone) +4 to +19 % with the small tiles, 2^26 elements (4.6 rounds) -1 to -28 %.
    if (fn != kCompressGeneral && tile_elems == kTileElems && !withhold_tile) {
        uint64_t std_tiles = 0;
        for (int k = 0; k < L; ++k) std_tiles += (st[k].n + kTileElems - 1) / kTileElems;
        if (std_tiles < kSmallCallTiles && 2 * std_tiles < 3 * (uint64_t)grid) {
            const void *const *from = compress_table(st[0].dt);
            const void *const *to = st[0].dt == LGN_BF16 ? kCompressTableBf16Small : kCompressTableF32Small;
            for (int v = 0; v < kVariants; ++v)
                if (from[v] == fn) { fn = to[v]; tile_elems = st[0].dt == LGN_BF16 ? kSmallTileElemsBf16 : kSmallTileElemsF32; break; }
            grid = persistent_ctas(fn);
            if (grid < 1) return LGN_ERR_CUDA;
        }
    }
    uint32_t partial0 = 0;
    for (int k = 0; k < L; ++k) {
        LayerState &s = st[k];
        s.ntiles = (uint32_t)((s.n + tile_elems - 1) / tile_elems);
        s.partial0 = partial0;
        partial0 += s.ntiles;
    }
    std::vector<Segment> segs;
    uint32_t total_items = 0;
    build_queue(st, segs, total_items, withhold_tile);
    {   // terminator so that the segment scan never runs off the table
        Segment s;
        memset(&s, 0, sizeof s);
        s.first_item = total_items; s.ntiles = 0xFFFFFFFFu - total_items;
        segs.push_back(s);
    }

    if (log_enabled()) {
        uint64_t elems = 0;
        for (int k = 0; k < L; ++k) elems += st[k].n;
        const int v = variant_of(st[0].mode, st[0].nbits, st[0].rounding);
        log_line("grouped call: %d layers, %llu elements; kernel: %s%s (variant %d of %s), tiles of %u elements, grid %d x %d threads, "
                 "%u queue items in %zu runs, counters %s, %d set-up launch(es), workspace %zu bytes",
                 L, (unsigned long long)elems, fn == kCompressGeneral ? "general (layers differ)" : "specialised",
                 (fn != kCompressGeneral && any_ext) ? " with extended statistics" : "", v, st[0].dt == LGN_BF16 ? "bf16" : "fp32",
                 tile_elems, grid, kThreads, total_items, segs.size() - 1, st[0].counters ? "on" : "off",
                 upload_launches(upload_bytes(w, L)), (size_t)w.total);
    }

    // image of [header | states | dyn (zero) | segments]
    std::vector<unsigned char> image(w.partials, 0);
    {
        WsHeader h;
        memset(&h, 0, sizeof h);
        h.weyl.w0 = kWeyl0; h.weyl.w1 = kWeyl1;
        memcpy(image.data(), &h, sizeof h);
    }
    memcpy(image.data() + w.states, st.data(), sizeof(LayerState) * (size_t)L);
    memcpy(image.data() + w.segs, segs.data(), sizeof(Segment) * segs.size());
    const size_t used = upload_bytes(w, L);
    unsigned char *base = static_cast<unsigned char *>(ws);
    if (used <= (size_t)kBlobBytes) upload_image<kBlobBytes>(image.data(), used, base, stream);
    else                            upload_image<kBigBlobBytes>(image.data(), used, base, stream);
    if (cudaGetLastError() != cudaSuccess) return LGN_ERR_CUDA;

    if ((uint32_t)grid > total_items) grid = (int)(total_items ? total_items : 1u);
    WsHeader *a_hdr = reinterpret_cast<WsHeader *>(base);
    const LayerState *a_states = reinterpret_cast<const LayerState *>(base + w.states);
    LayerDyn *a_dyn = reinterpret_cast<LayerDyn *>(base + w.dyn);
    const Segment *a_segs = reinterpret_cast<const Segment *>(base + w.segs);
    int a_L = L;
    uint32_t a_items = total_items;
    Partial *a_partials = reinterpret_cast<Partial *>(base + w.partials);
    void *args[] = { &a_hdr, &a_states, &a_dyn, &a_segs, &a_L, &a_items, &a_partials };
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;     // overlap the launch with the set-up launch before it
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelExC(&cfg, fn, args) != cudaSuccess) return LGN_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? LGN_OK : LGN_ERR_CUDA;
}

}  // namespace lgn

// ==================================================================== C ABI
using namespace lgn;

extern "C" const char *lgn_status_string(lgn_status s) {
    switch (s) {
        case LGN_OK: return "ok";
        case LGN_ERR_INVALID_ARG: return "invalid argument";
        case LGN_ERR_UNSUPPORTED: return "unsupported size or bit width";
        case LGN_ERR_WORKSPACE: return "workspace too small";
        case LGN_ERR_CUDA: return "CUDA runtime error";
        case LGN_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

extern "C" size_t lgn_workspace_bytes(const uint64_t *n_per_layer, int num_layers) {
    WsLayout w;
    if (num_layers > 0 && n_per_layer == nullptr) return 0;
    if (!ws_layout(n_per_layer, num_layers, w)) return 0;
    return w.total;
}

extern "C" int lgn_launches_per_call(int num_layers) {
    if (num_layers <= 0) return 0;
    std::vector<uint64_t> ns((size_t)num_layers, 1);
    WsLayout w;
    if (!ws_layout(ns.data(), num_layers, w)) return 0;
    return upload_launches(upload_bytes(w, num_layers)) + 1;
}

extern "C" size_t lgn_codes_bytes(uint64_t n, int nbits) {
    if (nbits < 4 || nbits > 8) return 0;
    const uint64_t bytes = (n * (uint64_t)nbits + 7) / 8;
    return (size_t)((bytes + 3) / 4 * 4);
}

extern "C" lgn_status lgn_stats(const void *g, uint64_t n, lgn_dtype dt, lgn_stats_t *out_dev,
                                void *ws, size_t ws_bytes, void *stream) {
    if (out_dev == nullptr || !aligned16(out_dev)) return LGN_ERR_INVALID_ARG;
    InternalLayer il;
    memset(&il, 0, sizeof il);
    il.d.g = g; il.d.n = n; il.d.dt = dt; il.d.mode = kModeStatsOnly;
    il.stats_out = out_dev;
    return run_layers(std::vector<InternalLayer>(1, il), ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

extern "C" lgn_status lgn_combine_stats(const lgn_stats_t *parts, int nparts, lgn_stats_t *out) {
    if (out == nullptr || nparts < 0 || (nparts > 0 && parts == nullptr)) return LGN_ERR_INVALID_ARG;
    lgn_stats_t t;
    t.n = 0; t.nnz = 0; t.sum_ln = t.sum_ln2 = t.mu = t.sigma = 0.0;
    for (int k = 0; k < nparts; ++k) {
        if (parts[k].nnz > parts[k].n || !std::isfinite(parts[k].sum_ln) || !std::isfinite(parts[k].sum_ln2))
            return LGN_ERR_INVALID_ARG;
        t.n += parts[k].n; t.nnz += parts[k].nnz;
        t.sum_ln += parts[k].sum_ln; t.sum_ln2 += parts[k].sum_ln2;
    }
    if (t.nnz) {
        t.mu = t.sum_ln / (double)t.nnz;
        double var = t.sum_ln2 / (double)t.nnz - t.mu * t.mu;
        t.sigma = var > 0.0 ? sqrt(var) : 0.0;
    }
    *out = t;
    return LGN_OK;
}

extern "C" lgn_status lgn_threshold(double mu, double sigma, double zero_frac, double S, double *tau) {
    if (tau == nullptr) return LGN_ERR_INVALID_ARG;
    *tau = 0.0;
    if (!(S >= 0.0 && S < 1.0) || !(zero_frac >= 0.0 && zero_frac <= 1.0)) return LGN_ERR_INVALID_ARG;
    if (!std::isfinite(mu) || !(sigma >= 0.0) || !std::isfinite(sigma)) return LGN_ERR_INVALID_ARG;
    *tau = threshold_for(mu, sigma, zero_frac, S);
    log_line("threshold: mu=%.17g sigma=%.17g zero fraction=%.17g S=%.17g -> S'=%.17g tau=%.17g", mu, sigma, zero_frac, S,
             zero_frac < 1.0 ? (S - zero_frac) / (1.0 - zero_frac) : 0.0, *tau);
    return LGN_OK;
}

extern "C" double lgn_snap_threshold(double tau, lgn_dtype dt) {
    if (!(tau >= 0.0)) return NAN;
    if (dt == LGN_F32) return (double)snap_threshold_f32(tau);
    if (dt == LGN_BF16) return (double)snap_threshold_bf16(tau);
    return NAN;
}

extern "C" lgn_status lgn_fp_format(double mu, double sigma, int nbits, lgn_fp_format_t *fmt) {
    if (fmt == nullptr) return LGN_ERR_INVALID_ARG;
    if (nbits < 4 || nbits > 8) return LGN_ERR_UNSUPPORTED;
    if (!std::isfinite(mu) || !(sigma >= 0.0) || !std::isfinite(sigma)) return LGN_ERR_INVALID_ARG;
    choose_format(mu, sigma, nbits, *fmt);
    log_line("format: mu=%.17g sigma=%.17g nbits=%d -> 1-%d-%d, scale 2^%d", mu, sigma, nbits, fmt->exp_bits, fmt->man_bits, fmt->scale_exp);
    return LGN_OK;
}

extern "C" lgn_status lgn_cosine_similarity(double mu, double sigma, double k, double tau, double *cosine) {
    if (cosine == nullptr) return LGN_ERR_INVALID_ARG;
    *cosine = 0.0;
    if (!std::isfinite(mu) || !(sigma >= 0.0) || !std::isfinite(sigma) || !std::isfinite(k)) return LGN_ERR_INVALID_ARG;
    if (!(tau > 0.0) || !std::isfinite(tau)) return LGN_ERR_INVALID_ARG;
    const double s = clamp_sigma(sigma), u = log(tau) - mu;
    if (u > k * s) return LGN_ERR_INVALID_ARG;
    *cosine = cosine_similarity_of(u, s, k);
    return LGN_OK;
}

extern "C" lgn_status lgn_allocate_sparsity(const lgn_alloc_layer_t *layers, int num_layers, int num_deep,
                                            double S, double s_max, double *S_out, double *achieved) {
    if (num_layers < 0 || num_deep < 0 || num_deep > num_layers) return LGN_ERR_INVALID_ARG;
    if (num_layers > 0 && (layers == nullptr || S_out == nullptr)) return LGN_ERR_INVALID_ARG;
    if (!(S >= 0.0 && S < 1.0) || !(s_max >= S && s_max < 1.0)) return LGN_ERR_INVALID_ARG;
    double total = 0.0, deep_n = 0.0, deep_zeros = 0.0;
    for (int i = 0; i < num_layers; ++i) {
        const lgn_alloc_layer_t &a = layers[i];
        if (!(a.zero_frac >= 0.0 && a.zero_frac <= 1.0) || !(a.sigma >= 0.0) || !std::isfinite(a.sigma)) return LGN_ERR_INVALID_ARG;
        if (i < num_deep && (!std::isfinite(a.k) || !(a.min_cos <= 1.0))) return LGN_ERR_INVALID_ARG;
        total += (double)a.n;
    }
    for (int i = 0; i < num_deep; ++i) {
        const lgn_alloc_layer_t &a = layers[i];
        const double s = clamp_sigma(a.sigma), l = a.zero_frac;
        double Si = S;
        if (l < 1.0 && S > l) {                                   // otherwise nothing is pruned here at S
            double u = solve_threshold_u(s, (S - l) / (1.0 - l));
            if (u > a.k * s) u = a.k * s;
            if (cosine_similarity_of(u, s, a.k) < a.min_cos) {    // below its floor: lower the threshold
                const double u2 = threshold_u_for_cosine(a.min_cos, s, a.k);
                double F, dF;
                pruned_fraction(u2, s, F, dF);
                Si = l + (1.0 - l) * F;
                if (Si > S) Si = S;
            }
        }
        S_out[i] = Si;
        deep_n += (double)a.n;
        deep_zeros += (double)a.n * Si;
    }
    double S_rest = S;
    const double rest_n = total - deep_n;
    if (rest_n > 0.0) {
        S_rest = (S * total - deep_zeros) / rest_n;
        if (S_rest > s_max) S_rest = s_max;
        if (S_rest < S) S_rest = S;
    }
    double zeros = deep_zeros;
    for (int i = num_deep; i < num_layers; ++i) { S_out[i] = S_rest; zeros += (double)layers[i].n * S_rest; }
    if (achieved) *achieved = total > 0.0 ? zeros / total : 0.0;
    return LGN_OK;
}

extern "C" lgn_status lgn_scale_from_max(double max_abs, int exp_bits, int32_t *scale_exp) {
    if (scale_exp == nullptr) return LGN_ERR_INVALID_ARG;
    if (!(max_abs > 0.0) || !std::isfinite(max_abs) || exp_bits < 1 || exp_bits > 7) return LGN_ERR_INVALID_ARG;
    int ex = 0;
    (void)std::frexp(max_abs, &ex);                          // max_abs = f 2^ex, f in [1/2, 1)
    *scale_exp = (ex - 1) - ((1 << (exp_bits - 1)) - 1);
    return LGN_OK;
}

static int apply_grid(const void *fn, uint32_t ntiles) {
    int g = persistent_ctas(fn);
    if (g < 1) return -1;
    return (uint32_t)g > ntiles ? (int)ntiles : g;
}

extern "C" lgn_status lgn_prune(const void *g, void *out, uint64_t n, lgn_dtype dt, double tau,
                                uint64_t seed, void *stream) {
    lgn_layer_t d;
    memset(&d, 0, sizeof d);
    d.g = g; d.out = out; d.n = n; d.dt = dt; d.mode = LGN_MODE_PRUNE; d.S = 0.0;
    lgn_status s = check_layer(d);
    if (s != LGN_OK) return s;
    if (!(tau >= 0.0)) return LGN_ERR_INVALID_ARG;
    if (n > (1ull << 44)) return LGN_ERR_UNSUPPORTED;
    if (n == 0) return LGN_OK;
    const uint32_t ntiles = (uint32_t)((n + kTileElems - 1) / kTileElems);
    const void *fn = kPruneTable[dt];
    const int grid = apply_grid(fn, ntiles);
    if (grid < 1) return LGN_ERR_CUDA;
    float tau_used = dt == LGN_BF16 ? snap_threshold_bf16(tau) : snap_threshold_f32(tau);
    uint32_t a_ntiles = ntiles;
    Weyl wy = { kWeyl0, kWeyl1 };
    void *args[] = { &g, &out, &n, &a_ntiles, &tau_used, &seed, &wy };
    if (cudaLaunchKernel(fn, dim3((unsigned)grid), dim3(kThreads), args, 0, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return LGN_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? LGN_OK : LGN_ERR_CUDA;
}

extern "C" lgn_status lgn_quantize(const void *g, void *codes, uint64_t n, lgn_dtype dt,
                                   const lgn_fp_format_t *fmt, lgn_rounding rounding,
                                   uint64_t seed, void *stream) {
    if (fmt == nullptr) return LGN_ERR_INVALID_ARG;
    if (fmt->nbits < 4 || fmt->nbits > 8) return LGN_ERR_UNSUPPORTED;
    if (fmt->exp_bits < 1 || fmt->man_bits < 0 || 1 + fmt->exp_bits + fmt->man_bits != fmt->nbits)
        return LGN_ERR_INVALID_ARG;
    if (fmt->scale_exp < -400 || fmt->scale_exp > 400) return LGN_ERR_INVALID_ARG;
    lgn_layer_t d;
    memset(&d, 0, sizeof d);
    d.g = g; d.out = codes; d.n = n; d.dt = dt; d.mode = LGN_MODE_QUANTIZE; d.nbits = fmt->nbits;
    d.rounding = rounding;
    lgn_status s = check_layer(d);
    if (s != LGN_OK) return s;
    if (n > (1ull << 44)) return LGN_ERR_UNSUPPORTED;
    if (n == 0) return LGN_OK;
    const uint32_t ntiles = (uint32_t)((n + kTileElems - 1) / kTileElems);
    const void *fn = kQuantizeTable[dt][2 * (fmt->nbits - 4) + (rounding == LGN_ROUND_STOCHASTIC ? 1 : 0)];
    const int grid = apply_grid(fn, ntiles);
    if (grid < 1) return LGN_ERR_CUDA;
    QuantParams q = make_quant_params(*fmt);
    uint32_t a_ntiles = ntiles;
    Weyl wy = { kWeyl0, kWeyl1 };
    void *args[] = { &g, &codes, &n, &a_ntiles, &q, &seed, &wy };
    if (cudaLaunchKernel(fn, dim3((unsigned)grid), dim3(kThreads), args, 0, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return LGN_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? LGN_OK : LGN_ERR_CUDA;
}

extern "C" lgn_status lgn_compress_layers(const lgn_layer_t *layers, int num_layers,
                                          lgn_layer_result_t *results_dev,
                                          void *ws, size_t ws_bytes, void *stream) {
    if (num_layers < 0) return LGN_ERR_INVALID_ARG;
    if (num_layers == 0) return LGN_OK;
    if (layers == nullptr || results_dev == nullptr || !aligned8(results_dev)) return LGN_ERR_INVALID_ARG;
    std::vector<InternalLayer> v((size_t)num_layers);
    for (int k = 0; k < num_layers; ++k) {
        if (layers[k].mode != LGN_MODE_PRUNE && layers[k].mode != LGN_MODE_QUANTIZE) return LGN_ERR_INVALID_ARG;
        v[k].d = layers[k];
        v[k].stats_out = nullptr;
        v[k].result_out = results_dev + k;
    }
    return run_layers(v, ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

extern "C" lgn_status lgn_selftest_wait_expires(const lgn_layer_t *layers, int num_layers,
                                                lgn_layer_result_t *results_dev,
                                                void *ws, size_t ws_bytes, void *stream) {
    if (num_layers <= 0 || layers == nullptr || results_dev == nullptr || !aligned8(results_dev))
        return LGN_ERR_INVALID_ARG;
    std::vector<InternalLayer> v((size_t)num_layers);
    for (int k = 0; k < num_layers; ++k) {
        if (layers[k].mode != LGN_MODE_PRUNE && layers[k].mode != LGN_MODE_QUANTIZE) return LGN_ERR_INVALID_ARG;
        v[k].d = layers[k];
        v[k].stats_out = nullptr;
        v[k].result_out = results_dev + k;
    }
    if (layers[0].n == 0) return LGN_ERR_INVALID_ARG;
    return run_layers(v, ws, ws_bytes, static_cast<cudaStream_t>(stream), true);
}

// ------------------------------------------------------------------ statistics without a caller workspace
// Scratch of lgn_stats_static_scratch: part of the library image on every device
// that loads it.  In host code this name is only a handle for the symbol, not an
// address a kernel can use: the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_stats_static_scratch[LGN_STATS_STATIC_SCRATCH_BYTES];

namespace {
// Device address of the array on the current device, looked up once per device
// (ordinals 0..63; host threads that make the first call together take turns).
void *static_scratch_address() {
    static void *cached[64];
    static std::mutex guard;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(guard);
    if (cached[dev] == nullptr) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_stats_static_scratch) != cudaSuccess) return nullptr;
        cached[dev] = p;
    }
    return cached[dev];
}
}  // namespace

extern "C" lgn_status lgn_stats_static_scratch(const void *g, uint64_t n, lgn_dtype dt, lgn_stats_t *out_dev,
                                               void *stream) {
    if (out_dev == nullptr || !aligned16(out_dev)) return LGN_ERR_INVALID_ARG;
    if (n > LGN_STATS_STATIC_MAX_ELEMS) return LGN_ERR_UNSUPPORTED;
    WsLayout w;
    if (!ws_layout(&n, 1, w) || w.total > sizeof(g_stats_static_scratch)) return LGN_ERR_UNSUPPORTED;
    InternalLayer il;
    memset(&il, 0, sizeof il);
    il.d.g = g; il.d.n = n; il.d.dt = dt; il.d.mode = kModeStatsOnly;
    il.stats_out = out_dev;
    lgn_status s = check_layer(il.d);                 // argument errors before touching CUDA
    if (s != LGN_OK) return s;
    void *scratch = static_scratch_address();
    if (scratch == nullptr) return LGN_ERR_CUDA;
    // run_layers rewrites the queue header, descriptors and counters on the stream
    // before the kernel reads them; partial sums are written before they are read.
    return run_layers(std::vector<InternalLayer>(1, il), scratch, sizeof(g_stats_static_scratch),
                      static_cast<cudaStream_t>(stream));
}
