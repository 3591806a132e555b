// One-shot statistics for callers that may not allocate device memory: the partial-statistics scratch of the
// accumulation lives in a fixed array that is part of the library image.
#include <mutex>

#include "cb_internal.cuh"

namespace cb {

// Built-in scratch: partial slots and the head-match tables.  Every GPU that loads the library
// holds this array until the process exits.
static constexpr size_t STATIC_SCRATCH_BYTES = (size_t)CB_STATIC_SCRATCH_MAX_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

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
    // the same host-side checks as cb_create + cb_stats_accumulate
    cb_status cs = check_problem(prob);
    if (cs != CB_OK) return cs;
    if (!G || !C) return CB_ERR_INVALID_ARG;
    const int d = prob->ds;
    cs = check_view(src, prob->Ls, prob->Hs, d);
    if (cs != CB_OK) return cs;
    cs = check_view(tgt, prob->Lt, prob->Ht, d);
    if (cs != CB_OK) return cs;
    const int64_t T = src->n_tokens;
    if (T <= 0 || T != tgt->n_tokens) return CB_ERR_INVALID_ARG;
    if (!w_k || !w_v || w_stride_layer < 0 || w_stride_head < 0) return CB_ERR_INVALID_ARG;
    if (((uintptr_t)w_k | (uintptr_t)w_v) & 3) return CB_ERR_INVALID_ARG;

    // layout inside the built-in array: [slots][tables]
    const int n_splits = prob->n_splits > 0 ? prob->n_splits : 1;
    const size_t n_maps = 2 * (size_t)prob->Lt * prob->Ht;
    const size_t slots_bytes = (size_t)n_splits * n_maps * slot_floats(d) * sizeof(float);
    const size_t tab_off = (slots_bytes + 255) / 256 * 256;
    const size_t end_off = (tab_off + sizeof(int) * ((size_t)prob->Lt + prob->Ht) + 255) / 256 * 256;
    if (end_off + 256 > STATIC_SCRATCH_BYTES) return CB_ERR_STATIC_LIMIT;

    unsigned char *base = nullptr;
    if (static_scratch_address(&base) != cudaSuccess) { return cuda_failed(); }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: everything that must start at zero is cleared here
    cudaError_t e = cudaMemsetAsync(base, 0, slots_bytes, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(base + tab_off, prob->src_layer, sizeof(int) * (size_t)prob->Lt, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(base + tab_off + sizeof(int) * (size_t)prob->Lt, prob->src_head, sizeof(int) * (size_t)prob->Ht,
                            cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_failed(e);

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
    a.status = library_status_word();     // a device-side time-out shows in cb_last_device_status
    const TestHooks hk = test_hooks();
    a.poll_limit = hk.poll_limit; a.starve = hk.starve;
    a.compensated = (prob->flags & CB_FLAG_COMPENSATED) ? 1 : 0;
    e = (prob->flags & CB_FLAG_SIMT) ? launch_accum_simt(a, d, st) : launch_accum_tc(a, d, src, tgt, st);
    if (e == cudaSuccess) e = launch_reduce(a.slots, n_splits, (int)n_maps, d, G, C, st);
    if (e != cudaSuccess) return cuda_failed(e);
    return CB_OK;
}
