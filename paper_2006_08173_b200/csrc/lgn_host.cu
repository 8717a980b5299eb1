// The grouped path for tensors that live in host memory (lgn_compress_layers_host).
//
// The layers are taken in groups of consecutive layers (at least kGroupBytes of input
// each).  Three streams run as a pipeline: the copies of group k+1 into the device
// buffer, the kernels of group k (one lgn_compress_layers call, on the caller's
// stream), and the copies of group k-1's outputs and results back, so that the two
// directions of the host link are busy at the same time and the kernels hide behind
// them.  Every layer has its own input and output region in the device buffer; the
// workspace is shared by the groups, which run one after the other on one stream.
#include <cstdint>
#include <vector>

#include <cuda_runtime.h>

#include "lgn.h"

namespace {

constexpr size_t kGroupBytes = 64u << 20;

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct StagingPlan {
    std::vector<size_t> in_off, out_off, mask_off, in_bytes, out_bytes;
    size_t results_off = 0, ws_off = 0, ws_bytes = 0, total = 0;
};

bool plan_staging(const lgn_layer_t *layers, int L, StagingPlan &p) {
    size_t off = 0;
    std::vector<uint64_t> ns((size_t)L);
    p.in_off.resize(L); p.out_off.resize(L); p.mask_off.resize(L); p.in_bytes.resize(L); p.out_bytes.resize(L);
    for (int k = 0; k < L; ++k) {
        const lgn_layer_t &d = layers[k];
        if (d.dt != LGN_F32 && d.dt != LGN_BF16) return false;
        if (d.mode == LGN_MODE_QUANTIZE && (d.nbits < 4 || d.nbits > 8)) return false;
        if (d.mode != LGN_MODE_QUANTIZE && d.mode != LGN_MODE_PRUNE) return false;
        ns[k] = d.n;
        p.in_bytes[k] = (size_t)d.n * (d.dt == LGN_BF16 ? 2u : 4u);
        p.out_bytes[k] = d.mode == LGN_MODE_PRUNE ? p.in_bytes[k] : lgn_codes_bytes(d.n, d.nbits);
        p.in_off[k] = off;  off += round_up(p.in_bytes[k], 256);
        p.out_off[k] = off; off += round_up(p.out_bytes[k], 256);
        p.mask_off[k] = off; if (d.right_mode) off += round_up((size_t)d.n, 256);
    }
    p.results_off = off; off += round_up(sizeof(lgn_layer_result_t) * (size_t)L, 256);
    p.ws_bytes = lgn_workspace_bytes(ns.data(), L);          // enough for every subset of the layers
    if (p.ws_bytes == 0) return false;
    p.ws_off = off; off += p.ws_bytes;
    p.total = off;
    return true;
}

// Streams and events of one call; released whatever way the call ends.
struct Pipeline {
    cudaStream_t in = nullptr, out = nullptr;
    std::vector<cudaEvent_t> events;
    bool ok = true;
    Pipeline() {
        ok = cudaStreamCreateWithFlags(&in, cudaStreamNonBlocking) == cudaSuccess &&
             cudaStreamCreateWithFlags(&out, cudaStreamNonBlocking) == cudaSuccess;
    }
    cudaEvent_t event() {
        cudaEvent_t e = nullptr;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { ok = false; return nullptr; }
        events.push_back(e);
        return e;
    }
    ~Pipeline() {
        if (in) { cudaStreamSynchronize(in); cudaStreamDestroy(in); }
        if (out) { cudaStreamSynchronize(out); cudaStreamDestroy(out); }
        for (cudaEvent_t e : events) cudaEventDestroy(e);
    }
};

}  // namespace

extern "C" size_t lgn_host_staging_bytes(const lgn_layer_t *layers, int num_layers) {
    if (num_layers <= 0 || layers == nullptr) return 0;
    StagingPlan p;
    return plan_staging(layers, num_layers, p) ? p.total : 0;
}

extern "C" lgn_status lgn_compress_layers_host(const lgn_layer_t *layers, int num_layers,
                                               lgn_layer_result_t *results_host,
                                               void *dev_buf, size_t dev_bytes, void *stream) {
    if (num_layers < 0) return LGN_ERR_INVALID_ARG;
    if (num_layers == 0) return LGN_OK;
    if (layers == nullptr || results_host == nullptr || dev_buf == nullptr) return LGN_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(dev_buf) & 255u) != 0) return LGN_ERR_INVALID_ARG;
    StagingPlan p;
    if (!plan_staging(layers, num_layers, p)) return LGN_ERR_INVALID_ARG;
    if (dev_bytes < p.total) return LGN_ERR_WORKSPACE;
    for (int k = 0; k < num_layers; ++k)
        if (layers[k].n > 0 && (layers[k].g == nullptr || layers[k].out == nullptr)) return LGN_ERR_INVALID_ARG;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *base = static_cast<char *>(dev_buf);
    std::vector<lgn_layer_t> dev_layers(layers, layers + num_layers);
    for (int k = 0; k < num_layers; ++k) {
        dev_layers[k].g = base + p.in_off[k];
        dev_layers[k].out = base + p.out_off[k];
        if (layers[k].right_mode) dev_layers[k].right_mode = base + p.mask_off[k];
    }
    lgn_layer_result_t *res_dev = reinterpret_cast<lgn_layer_result_t *>(base + p.results_off);

    Pipeline pipe;
    if (!pipe.ok) return LGN_ERR_CUDA;
    // the device buffer may still be in use by earlier work on the caller's stream
    cudaEvent_t start = pipe.event();
    if (!pipe.ok || cudaEventRecord(start, st) != cudaSuccess || cudaStreamWaitEvent(pipe.in, start, 0) != cudaSuccess)
        return LGN_ERR_CUDA;

    lgn_status status = LGN_OK;
    for (int first = 0; first < num_layers && status == LGN_OK;) {
        int last = first;                                        // group = layers [first, last]
        size_t bytes = p.in_bytes[first];
        while (last + 1 < num_layers && bytes < kGroupBytes) { ++last; bytes += p.in_bytes[last]; }
        const int count = last - first + 1;

        for (int k = first; k <= last; ++k) {                    // copies in
            if (p.in_bytes[k] &&
                cudaMemcpyAsync(base + p.in_off[k], layers[k].g, p.in_bytes[k], cudaMemcpyHostToDevice, pipe.in) != cudaSuccess)
                status = LGN_ERR_CUDA;
            if (layers[k].right_mode && layers[k].n &&
                cudaMemcpyAsync(base + p.mask_off[k], layers[k].right_mode, (size_t)layers[k].n, cudaMemcpyHostToDevice, pipe.in) != cudaSuccess)
                status = LGN_ERR_CUDA;
        }
        cudaEvent_t arrived = pipe.event(), computed = pipe.event();
        if (!pipe.ok || status != LGN_OK) { status = LGN_ERR_CUDA; break; }
        if (cudaEventRecord(arrived, pipe.in) != cudaSuccess || cudaStreamWaitEvent(st, arrived, 0) != cudaSuccess) { status = LGN_ERR_CUDA; break; }

        status = lgn_compress_layers(dev_layers.data() + first, count, res_dev + first, base + p.ws_off, p.ws_bytes, stream);
        if (status != LGN_OK) break;
        if (cudaEventRecord(computed, st) != cudaSuccess || cudaStreamWaitEvent(pipe.out, computed, 0) != cudaSuccess) { status = LGN_ERR_CUDA; break; }

        for (int k = first; k <= last; ++k)                      // copies out
            if (p.out_bytes[k] &&
                cudaMemcpyAsync(layers[k].out, base + p.out_off[k], p.out_bytes[k], cudaMemcpyDeviceToHost, pipe.out) != cudaSuccess)
                status = LGN_ERR_CUDA;
        if (cudaMemcpyAsync(results_host + first, res_dev + first, sizeof(lgn_layer_result_t) * (size_t)count,
                            cudaMemcpyDeviceToHost, pipe.out) != cudaSuccess)
            status = LGN_ERR_CUDA;
        first = last + 1;
    }
    // everything has landed when the three streams have drained (also on the error paths)
    const bool drained = cudaStreamSynchronize(pipe.in) == cudaSuccess && cudaStreamSynchronize(st) == cudaSuccess &&
                         cudaStreamSynchronize(pipe.out) == cudaSuccess;
    if (status != LGN_OK) return status;
    return drained ? LGN_OK : LGN_ERR_CUDA;
}
