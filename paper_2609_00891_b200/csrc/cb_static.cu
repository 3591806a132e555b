// One-shot statistics for callers that may not allocate device memory: the partial-statistics scratch of the
// accumulation lives in a fixed array that is part of the library image.
#include <mutex>

#include "cb_internal.cuh"

namespace cb {

// Built-in scratch: partial slots, the head-match tables and a status word.  Every GPU that loads the library
// holds this array until the process exits.
static constexpr size_t STATIC_SCRATCH_BYTES = (size_t)CB_STATIC_SCRATCH_MAX_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

static constexpr int MAX_DEVICES = 64;
static std::mutex g_static_mutex;
static unsigned char *g_static_ptr[MAX_DEVICES];   // device address of the array, per device, filled on first use

// In host code the array's name is only a stand-in: the device address has to be asked for, with the device
// that will run the kernels current.
static cudaError_t static_scratch_address(unsigned char **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_static_ptr[dev] = static_cast<unsigned char *>(p);
    }
    *out = g_static_ptr[dev];
    return cudaSuccess;
}

}  // namespace cb

using namespace cb;

extern "C" cb_status cb_stats_build_static(const cb_problem *prob, const cb_kv_view *src, const cb_kv_view *tgt,
                                           const float *w_k, const float *w_v,
                                           int64_t w_stride_layer, int64_t w_stride_head,
                                           float *G, float *C, void *stream)
{
    if (!prob || !prob->src_layer || !prob->src_head || !src || !tgt || !G || !C) return CB_ERR_INVALID_ARG;
    if (prob->Ls <= 0 || prob->Hs <= 0 || prob->Lt <= 0 || prob->Ht <= 0) return CB_ERR_INVALID_ARG;
    if (prob->ds != prob->dt || (prob->ds != 64 && prob->ds != 128)) return CB_ERR_UNSUPPORTED;
    if (prob->n_splits < 0 || prob->n_splits > 64) return CB_ERR_INVALID_ARG;
    for (int l = 0; l < prob->Lt; ++l)
        if (prob->src_layer[l] < 0 || prob->src_layer[l] >= prob->Ls) return CB_ERR_INVALID_ARG;
    for (int h = 0; h < prob->Ht; ++h)
        if (prob->src_head[h] < 0 || prob->src_head[h] >= prob->Hs) return CB_ERR_INVALID_ARG;
    const int d = prob->ds;
    if (src->n_layers != prob->Ls || src->n_heads != prob->Hs || src->head_dim != d) return CB_ERR_INVALID_ARG;
    if (tgt->n_layers != prob->Lt || tgt->n_heads != prob->Ht || tgt->head_dim != d) return CB_ERR_INVALID_ARG;
    const int64_t T = src->n_tokens;
    if (T <= 0 || T != tgt->n_tokens || T >= (1ll << 31)) return CB_ERR_INVALID_ARG;
    if (!src->k || !src->v || !tgt->k || !tgt->v || !w_k || !w_v) return CB_ERR_INVALID_ARG;
    if (((uintptr_t)src->k | (uintptr_t)src->v | (uintptr_t)tgt->k | (uintptr_t)tgt->v) & 15) return CB_ERR_INVALID_ARG;
    if ((src->stride_layer | src->stride_token | src->stride_head | tgt->stride_layer | tgt->stride_token | tgt->stride_head) & 7)
        return CB_ERR_INVALID_ARG;
    if (src->stride_token <= 0 || tgt->stride_token <= 0 || w_stride_layer < 0 || w_stride_head < 0) return CB_ERR_INVALID_ARG;

    // layout inside the built-in array: [slots][tables][status]
    const int n_splits = prob->n_splits > 0 ? prob->n_splits : 1;
    const size_t n_maps = 2 * (size_t)prob->Lt * prob->Ht;
    const size_t slots_bytes = (size_t)n_splits * n_maps * slot_floats(d) * sizeof(float);
    const size_t tab_off = (slots_bytes + 255) / 256 * 256;
    const size_t status_off = (tab_off + sizeof(int) * ((size_t)prob->Lt + prob->Ht) + 255) / 256 * 256;
    if (status_off + 256 > STATIC_SCRATCH_BYTES) return CB_ERR_STATIC_LIMIT;

    unsigned char *base = nullptr;
    if (static_scratch_address(&base) != cudaSuccess) { cudaGetLastError(); return CB_ERR_CUDA; }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: everything that must start at zero is cleared here
    cudaError_t e = cudaMemsetAsync(base, 0, slots_bytes, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(base + status_off, 0, 256, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(base + tab_off, prob->src_layer, sizeof(int) * (size_t)prob->Lt, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(base + tab_off + sizeof(int) * (size_t)prob->Lt, prob->src_head, sizeof(int) * (size_t)prob->Ht,
                            cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) { cudaGetLastError(); return CB_ERR_CUDA; }

    AccumArgs a;
    a.src = KVPtr{static_cast<const __nv_bfloat16 *>(src->k), static_cast<const __nv_bfloat16 *>(src->v),
                  src->stride_layer, src->stride_token, src->stride_head};
    a.tgt = KVPtr{static_cast<const __nv_bfloat16 *>(tgt->k), static_cast<const __nv_bfloat16 *>(tgt->v),
                  tgt->stride_layer, tgt->stride_token, tgt->stride_head};
    a.w_k = w_k; a.w_v = w_v; a.w_sl = w_stride_layer; a.w_sh = w_stride_head;
    a.n_tokens = (int)T;
    a.Lt = prob->Lt; a.Ht = prob->Ht; a.n_splits = n_splits;
    a.src_layer = reinterpret_cast<const int *>(base + tab_off);
    a.src_head = a.src_layer + prob->Lt;
    a.slots = reinterpret_cast<float *>(base);
    a.status = reinterpret_cast<int *>(base + status_off);
    a.compensated = (prob->flags & CB_FLAG_COMPENSATED) ? 1 : 0;
    e = (prob->flags & CB_FLAG_SIMT) ? launch_accum_simt(a, d, st) : launch_accum_tc(a, d, src, tgt, st);
    if (e == cudaSuccess) e = launch_reduce(a.slots, n_splits, (int)n_maps, d, G, C, st);
    if (e != cudaSuccess) { cudaGetLastError(); return CB_ERR_CUDA; }
    return CB_OK;
}
