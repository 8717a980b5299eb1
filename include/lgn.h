/*
 * lgn.h -- C ABI of the lognormal neural-gradient compression library for
 * NVIDIA B200 (sm_100a).
 *
 * The library runs, per gradient tensor, the path of "Neural gradients are
 * near-lognormal: improved quantized and sparse training" (arXiv 2006.08173):
 *
 *   statistics of ln|g| over the nonzero entries  (Section 3; Appendix A.8, A.9 step 3)
 *     -> closed form: pruning threshold for a requested sparsity (Eq. 6-8; A.9 steps 1-2)
 *                  or n-bit floating-point split and scale       (Eq. 4; Algorithm 1)
 *     -> elementwise pass: stochastic pruning (Eq. 5) or FP quantisation (Eq. 1-2)
 *
 * Conventions that hold for every entry point
 *  - "device" pointers are CUDA device addresses on the current device, owned
 *    by the caller for the whole call and until the work enqueued on `stream`
 *    has finished.  "host" pointers are ordinary process memory, read or
 *    written before the call returns.
 *  - The library allocates no device memory and keeps no state between calls,
 *    except the entry points that say otherwise.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *    All device work is enqueued on it and the call returns without waiting.
 *  - Tensors are contiguous and are treated as flat arrays of n elements; the
 *    element index used for randomness is the flat index.
 *  - Gradient tensors (g, and out of a pruning call) must be 32-byte aligned;
 *    code streams, workspaces and a device lgn_stats_t (lgn_stats,
 *    lgn_stats_static_scratch) 16-byte aligned, arrays of lgn_layer_result_t 8-byte
 *    aligned.  Input and output buffers must not overlap.
 *  - Inputs must be finite, with magnitudes below 2^104 (about 2e31).  +0 and -0
 *    both count as zero.
 *  - Argument errors are found on the host and returned before anything is
 *    enqueued.  A CUDA error at enqueue time is returned as LGN_ERR_CUDA.
 *  - Same inputs, seed and arguments give bitwise the same outputs and the same
 *    statistics on every run.
 *  - With the environment variable LGN_LOG set (to anything but "" or "0"; read once
 *    per process) the host side prints its decisions to stderr, one line each,
 *    prefixed "[lgn] ": the kernel, tile size, grid and queue of a grouped call,
 *    the selection path of a quantile, the closed forms' inputs and results, the
 *    reason an argument was refused.  Device work is not affected.
 */
#ifndef LGN_H
#define LGN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LGN_OK              = 0,
    LGN_ERR_INVALID_ARG = 1,  /* null/misaligned pointer, S outside [0,1), bad enum, ... */
    LGN_ERR_UNSUPPORTED = 2,  /* nbits outside 4..8, tensor too large                     */
    LGN_ERR_WORKSPACE   = 3,  /* workspace smaller than lgn_workspace_bytes() says        */
    LGN_ERR_CUDA        = 4,  /* the CUDA runtime refused a launch or copy                */
    LGN_ERR_TIMEOUT     = 5   /* a bounded device-side wait ran out (per-layer status)    */
} lgn_status;

typedef enum { LGN_F32 = 0, LGN_BF16 = 1 } lgn_dtype;
typedef enum { LGN_ROUND_NEAREST = 0, LGN_ROUND_STOCHASTIC = 1 } lgn_rounding;
typedef enum { LGN_MODE_PRUNE = 0, LGN_MODE_QUANTIZE = 1 } lgn_mode;
/* Where a quantised layer's power-of-two scale comes from (Algorithm 1):
 *   LGN_SCALE_CENTRED   e_s = floor(mu/ln 2 + 1/2): the median magnitude sits in the middle
 *                       of the format's range, the setting Eq. 4 is derived for
 *   LGN_SCALE_FROM_MAX  e_s = floor(log2 max|g|) - (E_max - 1): the largest element sits in
 *                       the top binade, so nothing is clipped and the range is spent on the
 *                       large magnitudes at the expense of the smallest ones (the trade
 *                       described in the appendix "Gradient scaling") */
typedef enum { LGN_SCALE_CENTRED = 0, LGN_SCALE_FROM_MAX = 1 } lgn_scale_mode;

/* Lognormal statistics of one tensor (Section 3: magnitudes, zeros left out). */
typedef struct {
    uint64_t n;        /* elements                                               */
    uint64_t nnz;      /* elements != 0                                          */
    double   sum_ln;   /* sum of ln|g| over the nonzero elements                 */
    double   sum_ln2;  /* sum of (ln|g|)^2 over the same                         */
    double   mu;       /* sum_ln / nnz                      (0 when nnz == 0)    */
    double   sigma;    /* population standard deviation of ln|g| (0 when nnz==0) */
} lgn_stats_t;

/* An n-bit floating-point format: 1 sign bit, exp_bits, man_bits, and the
 * per-layer power-of-two scale of Algorithm 1 (values are divided by
 * 2^scale_exp before quantisation).  1 + exp_bits + man_bits == nbits. */
typedef struct {
    int32_t nbits;      /* 4..8                    */
    int32_t exp_bits;   /* n2, 1..nbits-1          */
    int32_t man_bits;   /* n1, 0..nbits-2          */
    int32_t scale_exp;  /* e_s                     */
} lgn_fp_format_t;

/* Text for a status code (static storage). */
const char *lgn_status_string(lgn_status s);

/* Device workspace, in bytes, that lgn_stats (num_layers = 1) or
 * lgn_compress_layers needs for tensors of these element counts.
 * n_per_layer: host.  Returns 0 if num_layers < 0 or a tensor is too large. */
size_t lgn_workspace_bytes(const uint64_t *n_per_layer, int num_layers);

/* Kernel launches one lgn_compress_layers call of num_layers tensors enqueues:
 * the set-up launches that carry the descriptors plus the one compute launch.
 * (lgn_stats: the value for 1 layer; lgn_prune / lgn_quantize: always 1.) */
int lgn_launches_per_call(int num_layers);

/* Bytes of the packed code stream of n codes of nbits each:
 * ceil(n*nbits/8) rounded up to a multiple of 4.  0 for nbits outside 4..8. */
size_t lgn_codes_bytes(uint64_t n, int nbits);

/* Statistics pass (Section 3; Appendix A.8 "mean and standard deviation of
 * the input", A.9 step 3): nnz, and the mean and population standard deviation
 * of the natural log of |g| over the nonzero elements.
 *   g        device, n elements of dt, read only
 *   out_dev  device, one lgn_stats_t, written when the stream reaches the call
 *   ws       device scratch of at least lgn_workspace_bytes(&n, 1) bytes;
 *            contents before and after are meaningless
 * The logarithm is evaluated in fp32 (base-2 hardware approximation), summed
 * in short fp32 runs and then in fp64, and combined across the grid in a fixed
 * order: deterministic, within 1e-5 relative of an fp64 evaluation.
 * n == 0 writes all zeros. */
lgn_status lgn_stats(const void *g, uint64_t n, lgn_dtype dt, lgn_stats_t *out_dev,
                     void *ws, size_t ws_bytes, void *stream);

/* Statistics of the union of several tensors from the statistics of each: n, nnz,
 * sum_ln and sum_ln2 add up; mu and sigma are formed from the totals.  This is the
 * one exchange step of data-parallel training that wants the SAME threshold or format
 * on every rank for a layer (each rank holds its own micro-batch slice of the
 * gradient): the ranks all-reduce these four sums per layer (32 bytes) between the
 * statistics pass and the closed form.  Host only.
 *   parts  host array of nparts records (their mu and sigma fields are ignored)
 *   out    host, receives the combined record */
lgn_status lgn_combine_stats(const lgn_stats_t *parts, int nparts, lgn_stats_t *out);

/* Sparsity -> threshold (Eq. 8 solved for alpha; Appendix A.9 steps 1-2).
 * Host only, no CUDA call.
 *   mu, sigma  lognormal parameters of the nonzero part
 *   zero_frac  l, fraction of the tensor that is exactly zero, in [0,1]
 *   S          requested fraction of zeros in the OUTPUT tensor, in [0,1)
 *   tau        host, receives alpha (fp64, not yet rounded to the tensor type)
 * The nonzero part has to reach S' = (S - l)/(1 - l); S' <= 0 or l == 1 gives
 * tau = 0 (no pruning).  sigma is clamped to [1e-6, 25]. */
lgn_status lgn_threshold(double mu, double sigma, double zero_frac, double S, double *tau);

/* The threshold as the pruning kernel holds it: tau rounded to the tensor's
 * storage type (ties to even; bf16 via fp32) and clamped to the largest finite
 * value.  Host only.  Returns NaN for a negative or NaN tau or a bad dtype. */
double lgn_snap_threshold(double tau, lgn_dtype dt);

/* Optimal exponent/mantissa split and scale (Eq. 4 minimised over the integer
 * splits n1 + n2 = nbits - 1, n2 >= 1; ties to the smaller n2) and the layer
 * scale e_s = floor(mu/ln 2 + 1/2).  Host only.  Eq. 4 is read with the
 * standard deviation of log2|g|, sigma/ln 2, and mantissa step 2^-n1.
 *   fmt  host, receives the format.  sigma is clamped to [1e-6, 25]. */
lgn_status lgn_fp_format(double mu, double sigma, int nbits, lgn_fp_format_t *fmt);

/* Algorithm 1's scale taken from the tensor's maximum, for a format with exp_bits
 * exponent bits: e_s = floor(log2 max_abs) - (2^(exp_bits-1) - 1).  Host only.
 * max_abs must be finite and > 0, exp_bits in 1..7. */
lgn_status lgn_scale_from_max(double max_abs, int exp_bits, int32_t *scale_exp);

/* ---- Cosine similarity and per-layer sparsity (appendix "Cosine similarity and
 * heterogeneous stochastic pruning") ----
 * lgn_cosine_similarity: the expected cosine of the angle between a layer's gradient and
 * its stochastically pruned copy at threshold tau, for magnitudes whose logarithm is
 * normal (mu, sigma) and cut off k standard deviations above mu (the appendix observes
 * that measured gradients lack the lognormal's far upper tail; k is the 0.997 quantile
 * of the data in sigmas, lgn_quantile).  Host only.  tau must be > 0 and ln(tau) - mu <= k*sigma
 * (a threshold above the cut prunes everything): otherwise LGN_ERR_INVALID_ARG. */
lgn_status lgn_cosine_similarity(double mu, double sigma, double k, double tau, double *cosine);

/* lgn_allocate_sparsity: the heterogeneous scheme.  Layers in backward-pass order,
 * deepest first; the first num_deep of them carry a floor min_cos on the expected
 * cosine similarity.  A deep layer whose cosine at the overall sparsity S is below its
 * floor gets the lower sparsity at which the floor is met; the remaining layers share
 * the one level that restores the element-weighted budget S, limited to s_max (the
 * appendix suggests 0.96-0.98) and not below S.  Host only.
 *   layers     host array; sigma, zero_frac, k of each layer from its statistics
 *   S_out      host array of num_layers sparsities, to be used as lgn_layer_t.S
 *   achieved   host, may be NULL: the element-weighted mean of S_out (below S when
 *              the cap binds) */
typedef struct {
    uint64_t n;          /* elements                                                  */
    double   sigma;      /* std of ln|g| over the nonzeros (clamped to [1e-6, 25])     */
    double   zero_frac;  /* l, fraction of exact zeros                                */
    double   k;          /* cut of the lognormal, in sigmas                            */
    double   min_cos;    /* floor on the cosine similarity (deep layers only)          */
} lgn_alloc_layer_t;
lgn_status lgn_allocate_sparsity(const lgn_alloc_layer_t *layers, int num_layers, int num_deep,
                                 double S, double s_max, double *S_out, double *achieved);

/* lgn_quantile: the order statistic of rank ceil(q * nnz) (1-based) of |g| over the
 * nonzero elements, exactly, by selection on the magnitude patterns.  With the layer's
 * mu and sigma, k = (ln(value) - mu) / sigma is the cut used above.
 *   g        device, n elements of dt, 32-byte aligned
 *   q        in [0, 1]
 *   out_dev  device, 16 bytes, 16-byte aligned: { float value; uint32_t pad; uint64_t nnz }
 *            (value 0 when the tensor has no nonzero element)
 *   ws       device scratch of lgn_quantile_workspace_bytes() bytes (4.5 MiB), 16-byte aligned
 * Tensors below 2^24 elements: radix selection, one read of a bf16 tensor, two of an fp32
 * tensor.  Larger tensors are read once (plus a sample of at least 2^21 elements): a
 * bracket around the wanted element is taken from the sample, the full read counts what
 * lies below it and sets aside what lies inside, and the answer is picked among those; if
 * the bracket turns out not to hold the element, or holds more than the scratch has room
 * for (2^16 fp32 patterns per sixteenth of the bracket; 4096 bf16 values), the radix
 * selection runs after all.  For fp32 and q far from 0 and 1 the sample needed grows with
 * n^2 q (1 - q); where it would pass n / 8 the radix selection is used at once.  The result
 * is exact in every case.
 * n must be below 2^32 (the histogram bins are 32-bit counters): a larger n returns
 * LGN_ERR_UNSUPPORTED and nothing is enqueued.
 * One memset and one to four launches on `stream`, no allocation. */
typedef struct { float value; uint32_t pad; uint64_t nnz; } lgn_quantile_t;
size_t     lgn_quantile_workspace_bytes(void);
lgn_status lgn_quantile(const void *g, uint64_t n, lgn_dtype dt, double q, lgn_quantile_t *out_dev,
                        void *ws, size_t ws_bytes, void *stream);

/* Stochastic pruning with a given threshold (Eq. 5): the steady-state call
 * between refreshes of the statistics.
 *   g, out  device, n elements of dt; out has the same type and layout
 *   tau     alpha >= 0; the kernel uses lgn_snap_threshold(tau, dt)
 *   seed    element i draws eps_i = (h_i + 1) / 2^16 in (0, 1] (Eq. 5's eps ~ U[0,1] on a
 *           grid of 2^16 points that leaves out 0, so that alpha*eps_i > 0 and a zero can
 *           never be kept), h_i = 16 bits of a Philox4x32-7 block: key = (seed low, seed
 *           high), counter = (i/8 low, i/8 high, 0, 0), word (i/2) mod 4, low half for
 *           even i, high half for odd i
 * |g_i| > alpha -> g_i;  fl32(alpha*eps_i) <= |g_i| <= alpha -> sign(g_i)*alpha;
 * otherwise +0.  Zeros stay +0.  An element with 0 < |g_i| <= alpha is kept with
 * probability floor(2^16 |g_i| / alpha) / 2^16 (up to the one rounding of alpha*eps_i),
 * so E[out_i] falls short of g_i by less than alpha * 2^-16; Eq. 5 with a continuous eps
 * is exactly unbiased. */
lgn_status lgn_prune(const void *g, void *out, uint64_t n, lgn_dtype dt, double tau,
                     uint64_t seed, void *stream);

/* FP quantisation with a given format (Eq. 1-2, Algorithm 1) into packed codes.
 *   g      device, n elements of dt
 *   codes  device, lgn_codes_bytes(n, fmt->nbits) bytes, all of them written:
 *          a little-endian bit stream, code i in bits [i*nbits, (i+1)*nbits),
 *          code = [sign | exponent field | mantissa], unused tail bits zero
 *   fmt    host
 *   seed   as in lgn_prune; used only with LGN_ROUND_STOCHASTIC
 * With x' = x / 2^scale_exp = M * 2^E, E_max = 2^(exp_bits-1):
 *   E >= E_max  (before rounding) -> largest code;
 *   E <= -E_max (before rounding) -> 0, under both roundings;
 *   else M rounded to man_bits (nearest: ties to the even mantissa; stochastic:
 *   h_i/2^16 of one mantissa step added, then truncated: the value rounds up with
 *   probability floor(frac * 2^16) / 2^16 for a dropped fraction frac, so the expected
 *   result falls short of x by less than 2^-16 of one mantissa step),
 *   a carry out of M moves to E, and E reaching E_max gives the largest code.
 * Exponent field = E + E_max (1..2^exp_bits-1); field 0 encodes zero.
 * A code decodes to (-1)^s (1 + m/2^man_bits) 2^(field - E_max + scale_exp). */
lgn_status lgn_quantize(const void *g, void *codes, uint64_t n, lgn_dtype dt,
                        const lgn_fp_format_t *fmt, lgn_rounding rounding,
                        uint64_t seed, void *stream);

/* One tensor of a grouped call. */
typedef struct {
    const void  *g;          /* device, n elements of dt                                  */
    void        *out;        /* device: n elements of dt (prune) or lgn_codes_bytes(n,nbits) */
    uint64_t     n;
    int32_t      dt;         /* lgn_dtype                                                  */
    int32_t      mode;       /* lgn_mode                                                   */
    double       S;          /* prune: requested output sparsity in [0,1)                  */
    int32_t      nbits;      /* quantize: 4..8                                             */
    int32_t      rounding;   /* quantize: lgn_rounding                                     */
    uint64_t     seed;
    int32_t      use_override;   /* nonzero: use mu_override/sigma_override in the closed  */
    int32_t      scale_mode;     /* form instead of the measured mu/sigma (nnz and the     */
    double       mu_override;    /* zero fraction are always the measured ones)            */
    double       sigma_override; /* scale_mode: quantize only, lgn_scale_mode; 0 for prune  */
    /* Bi-modal pruning (appendix "Algorithm for bi-modal lognormal pruning"), prune only,
     * NULL otherwise.  Device, n bytes, 16-byte aligned: byte i != 0 says that entry i
     * belongs to the RIGHT mode, i.e. that the same entry of the gradient after
     * batch-norm (the one the ReLU's backward produced) is non-zero; g itself is the
     * dense gradient before batch-norm.  With a mask, l is the fraction of left-mode
     * entries (step 1), mu and sigma are taken over the right-mode entries of g only
     * (step 3), S' = (S - l)/(1 - l) (step 2), and the threshold so obtained prunes the
     * WHOLE tensor (step 4). */
    const void  *right_mode;
    /* Nonzero: the apply pass also counts what it did to this layer (n_zero_out .. n_underflow
     * of the result record).  The counts cost the integer pipe a few instructions per element
     * (measured on B200: a call takes 10 % (fp32 FP6) to 30 % (bf16 pruning) longer), so they
     * are taken only when asked for: as soon as one layer of a call sets this field, every
     * layer of that call gets its counts (the call then runs through the second set of kernel
     * instances, the one that also serves right_mode and LGN_SCALE_FROM_MAX); a call whose
     * layers differ in type, mode, width or rounding always counts. */
    int32_t      counters;
    int32_t      reserved;   /* 0 */
} lgn_layer_t;

typedef struct {
    lgn_stats_t      stats;   /* measured, whatever the override says; with a right_mode   */
                              /* mask: nnz, sums, mu, sigma are over the right mode only    */
    double           tau;     /* prune: the threshold used (already snapped); else 0       */
    lgn_fp_format_t  fmt;     /* quantize: the format used; else zeros                     */
    int32_t          status;  /* lgn_status of this layer (LGN_ERR_TIMEOUT: output invalid) */
    float            max_abs; /* max|g| over the whole tensor; measured only for layers     */
                              /* with LGN_SCALE_FROM_MAX or a right_mode mask, else 0       */
    uint64_t         n_right_mode;  /* with a mask: entries whose mask byte != 0; else 0   */
    /* What the apply pass did (see lgn_layer_t.counters; all 0 when the call did not count):  */
    uint64_t         n_zero_out;    /* prune: output elements that are zero (achieved sparsity  */
                                    /* = n_zero_out / n); quantize: codes that are zero         */
    uint64_t         n_snapped;     /* prune: elements set to +-alpha (Eq. 5, middle case)      */
    uint64_t         n_saturated;   /* quantize: codes of the largest magnitude, where values    */
                                    /* at or beyond the top of the range land (Eq. 2, clip)      */
    uint64_t         n_underflow;   /* quantize: nonzero elements below the smallest normal,     */
                                    /* flushed to the zero code (Eq. 2, E <= -E_max)             */
} lgn_layer_result_t;

/* The whole path for a list of tensors in one kernel launch (plus one tiny
 * set-up launch): statistics -> closed form on the device -> apply, per layer,
 * with per-layer sparsity or bit-width (Section 5.3: different sparsity levels
 * at different layers).  Tiles of all layers go through one work queue; a
 * layer's apply tiles start as soon as its own statistics are complete, so a
 * tensor that fits in L2 is still there when it is read the second time.
 *   layers       host array of num_layers descriptors (copied before return)
 *   results_dev  device array of num_layers results
 *   ws           device scratch, lgn_workspace_bytes(n_per_layer, num_layers)
 * Device-side waits are bounded; if one runs out the layer's status is
 * LGN_ERR_TIMEOUT and the kernel still ends. */
lgn_status lgn_compress_layers(const lgn_layer_t *layers, int num_layers,
                               lgn_layer_result_t *results_dev,
                               void *ws, size_t ws_bytes, void *stream);

/* ---- Prefix code for pruned tensors (the paper's appendix "Encoding") ----------
 * Code words, emitted left to right: a zero -> "0", +alpha -> "100", -alpha ->
 * "101", any other value -> "11" followed by the value itself.  The paper gives
 * the table only; the container is this library's:
 *   - elements in index order, in blocks of LGN_PREFIX_BLOCK; block b occupies the
 *     32-bit words off[b] .. off[b+1]-1 of the stream (zero bits pad it to a whole
 *     word); off[nblocks] is the stream length in words;
 *   - stream bit k is bit (k mod 32) of word (k div 32);
 *   - the value after "11" is the element's own bit pattern (32 bits fp32, 16 bits
 *     bf16), least-significant bit first;
 *   - "0" stands for the pattern of +0 only (a -0 travels as a value: the code is
 *     lossless); the alpha codes are used only when alpha > 0.
 * lgn_prefix_encode reads g (device, 32-byte aligned, n elements).  With
 * apply_prune != 0 it first applies Eq. 5 with threshold alpha and `seed` to every
 * element on the fly -- bit for bit what lgn_prune would have written -- so the
 * dense pruned tensor never exists; with apply_prune == 0 g is taken as it is (an
 * already pruned tensor).  alpha is `tau` (snapped to the tensor's type like
 * lgn_prune does), or, if tau_from_dev is not NULL, the tau field of that
 * device-resident layer result (so that the call can follow lgn_compress_layers on
 * the same stream without a host round trip).
 * Outputs (device): off_dev[0 .. lgn_prefix_blocks(n)] and stream_dev.  A block
 * that would end beyond capacity_words is not written; the caller detects this
 * as off_dev[nblocks] > capacity_words.  lgn_prefix_bound_words(n, dt) is the
 * capacity that always suffices.  ws: device scratch of
 * lgn_prefix_workspace_bytes(n) bytes, 16-byte aligned, free again when the call's
 * work on `stream` has finished.  Errors: as for the other entry points; n above
 * 2^34 is LGN_ERR_UNSUPPORTED.  One memset of the workspace and one launch, no
 * allocation, no synchronisation.  Blocks obtain their first word from the lengths the
 * blocks before them have published; these device-side waits are bounded, and if one
 * runs out (it cannot while the GPU makes progress) off_dev[nblocks] is set to
 * 2^64 - 1, which the caller sees as "does not fit".
 * lgn_prefix_decode is the inverse: n elements of type dt into out_dev. */
#define LGN_PREFIX_BLOCK 2048u
uint64_t   lgn_prefix_blocks(uint64_t n);
uint64_t   lgn_prefix_bound_words(uint64_t n, lgn_dtype dt);
size_t     lgn_prefix_workspace_bytes(uint64_t n);
lgn_status lgn_prefix_encode(const void *g, uint64_t n, lgn_dtype dt, double tau, uint64_t seed,
                             int apply_prune, const lgn_layer_result_t *tau_from_dev,
                             uint32_t *stream_dev, uint64_t capacity_words, uint64_t *off_dev,
                             void *ws, size_t ws_bytes, void *stream);
lgn_status lgn_prefix_decode(const uint32_t *stream_dev, const uint64_t *off_dev, uint64_t n, lgn_dtype dt,
                             double tau, const lgn_layer_result_t *tau_from_dev, void *out_dev,
                             void *stream);

/* ---- Decoder of a packed code stream (Algorithm 1, last step: X_Q = 2^e_s * Q_FP) ----
 * What the consumer of a quantised gradient calls: code i of the stream written by
 * lgn_quantize or lgn_compress_layers becomes element i of a dense fp32 or bf16
 * tensor,  (-1)^s (1 + m / 2^man_bits) 2^(field - E_max + scale_exp)  for an
 * exponent field != 0 and +0 for field 0 (whatever its sign and mantissa bits).
 *   codes   device, lgn_codes_bytes(n, fmt->nbits) bytes, 16-byte aligned, read only
 *   fmt     host; the format the stream was written with
 *   out_dt  type of the output tensor (need not be the type that was quantised)
 *   out     device, n elements of out_dt, 32-byte aligned, must not overlap codes
 * Every value of a format has at most 7 significant bits, so the result is exact in
 * both output types as long as the format's exponents are normal fp32 exponents:
 * a format with 127 + scale_exp - E_max < 0 or scale_exp + E_max > 128 returns
 * LGN_ERR_UNSUPPORTED (nothing is enqueued).  One launch, no workspace. */
lgn_status lgn_dequantize(const void *codes, uint64_t n, const lgn_fp_format_t *fmt, lgn_dtype out_dt,
                          void *out, void *stream);

/* Self-test of the bounded device-side wait (no counterpart in the paper).
 * Same arguments and the same work as lgn_compress_layers, except that one
 * statistics tile of layer 0 is withheld from the queue, so layer 0's closed form
 * is never published.  Every apply tile of layer 0 must give up after the bounded
 * wait (about a second) instead of spinning for ever: the kernel ends,
 * results_dev[0].status becomes LGN_ERR_TIMEOUT (its output is not written), the
 * other layers complete normally, and the CUDA context stays usable.  results_dev
 * must be zero-filled by the caller (layer 0's record is otherwise untouched).
 * Nothing faults, traps or hangs.  layers[0].n must be > 0. */
lgn_status lgn_selftest_wait_expires(const lgn_layer_t *layers, int num_layers,
                                     lgn_layer_result_t *results_dev,
                                     void *ws, size_t ws_bytes, void *stream);

/* Statistics pass that needs no workspace from the caller.  (The paper has no
 * counterpart: this is a convenience of the library, not a step of the method.)
 *
 * Same result as lgn_stats, bit for bit.  It is meant for callers that cannot
 * allocate device memory at the point of the call: a hook that runs in the
 * middle of a training step, where cudaMalloc would synchronise the whole
 * device; a process that gave all free device memory to its own pool at start-up,
 * so that a later cudaMalloc fails; a C or C++ plug-in that has no access to the
 * host framework's allocator.  Such a caller still owns g and out_dev, but the
 * kernel's scratch (queue header, descriptors, per-tile partial sums) lives in
 * an array of LGN_STATS_STATIC_SCRATCH_BYTES bytes that is part of the library
 * image: every GPU that loads the library holds it from load to process exit.
 *   g, n, dt, out_dev, stream   as for lgn_stats
 *   n above LGN_STATS_STATIC_MAX_ELEMS returns LGN_ERR_UNSUPPORTED (nothing is
 *   enqueued); use lgn_stats with a caller workspace for larger tensors.
 * The call itself allocates nothing on the device, neither directly nor through
 * a library.  The first call on each device looks up the array's device address
 * (one cudaGetSymbolAddress, with that device current) and remembers it; make
 * that first call before starting any stream capture.  The look-up is serialised
 * among host threads, and serves device ordinals 0..63: on a device with a higher
 * ordinal the call returns LGN_ERR_CUDA and enqueues nothing.
 * All calls on one device share the one array: it still holds the previous
 * call's contents when the next call starts (the call re-initialises what it
 * reads), and two calls whose kernels can overlap on the GPU -- different
 * streams without an ordering between them -- race on it and give wrong
 * statistics.  Calls on one stream, or ordered by events, are safe. */
#define LGN_STATS_STATIC_MAX_ELEMS      (1ull << 28)
#define LGN_STATS_STATIC_SCRATCH_BYTES  (1024u + 32u * (1u << 14))
lgn_status lgn_stats_static_scratch(const void *g, uint64_t n, lgn_dtype dt, lgn_stats_t *out_dev,
                                    void *stream);

/* The grouped path for tensors that live in HOST memory: copies every input to
 * the device, runs lgn_compress_layers, copies every output and the results
 * back, and waits until all of it has landed.  The layers go through in groups of
 * consecutive layers (about 64 MB of input each) on three streams (the caller's for
 * the kernels, two that the call creates and destroys for the copies), so that
 * copies in, kernels and copies out of neighbouring groups overlap; each layer's
 * output and result are those of the single grouped call.  This is the end-to-end form of the call a
 * training loop on another device (or a test harness) makes; the paper's own
 * setting keeps the gradients on the accelerator and needs no copy.
 *   layers        host array; g and out of each entry are HOST pointers
 *                 (page-locked memory lets the copies run at full PCIe rate)
 *   results_host  host array of num_layers results
 *   dev_buf       device scratch of at least lgn_host_staging_bytes(layers,
 *                 num_layers) bytes, 256-byte aligned; holds the device copies
 *                 of inputs and outputs, the results and the workspace
 * Returns after the three streams have drained. */
size_t lgn_host_staging_bytes(const lgn_layer_t *layers, int num_layers);
lgn_status lgn_compress_layers_host(const lgn_layer_t *layers, int num_layers,
                                    lgn_layer_result_t *results_host,
                                    void *dev_buf, size_t dev_bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* LGN_H */
