// Per-device host state shared by the launchers: SM counts, the library's own device status word (for the entry
// points that have no context to carry one) and the test hooks that make a bounded device-side wait run out.
#include <atomic>
#include <mutex>

#include "cb_internal.cuh"

namespace cb {

// Set to DEV_TIMEOUT by any kernel launched without a context whose bounded wait ran out; read and cleared by
// cb_last_device_status.  One word per GPU that loads the library.
static __device__ int g_status_word;

static std::mutex g_mutex;
static int *g_status_ptr[MAX_DEVICES];
static int g_sm_count[MAX_DEVICES];
static std::atomic<unsigned> g_poll_limit{1u << 22};
static std::atomic<int> g_starve{0};

static int current_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return -1; }
    return (dev >= 0 && dev < MAX_DEVICES) ? dev : -1;
}

int device_sm_count()
{
    const int dev = current_device();
    if (dev < 0) return 148;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_sm_count[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) { cudaGetLastError(); n = 148; }
        g_sm_count[dev] = n;
    }
    return g_sm_count[dev];
}

// In host code the variable's name is a stand-in, not a device address: ask for the address with the device current.
int *library_status_word()
{
    const int dev = current_device();
    if (dev < 0) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_status_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        g_status_ptr[dev] = static_cast<int *>(p);
    }
    return g_status_ptr[dev];
}

TestHooks test_hooks() { return TestHooks{g_poll_limit.load(), g_starve.load()}; }

static std::atomic<int> g_last_cuda_error{0};

cb_status cuda_failed(cudaError_t e)
{
    const cudaError_t last = cudaGetLastError();     // also clears the runtime's (non-sticky) last-error state
    if (e == cudaSuccess) e = last;
    if (e == cudaSuccess) e = cudaErrorUnknown;
    g_last_cuda_error.store((int)e);
    return CB_ERR_CUDA;
}

}  // namespace cb

using namespace cb;

extern "C" cb_status cb_last_device_status(void *stream)
{
    int *w = library_status_word();
    if (!w) return cuda_failed(cudaErrorNoDevice);      // no current device, or its symbol address was refused
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int h = 0;
    cudaError_t e = cudaMemcpyAsync(&h, w, sizeof h, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && (e = cudaStreamSynchronize(st)) == cudaSuccess && h != DEV_OK) {
        e = cudaMemsetAsync(w, 0, sizeof h, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    }
    if (e != cudaSuccess) return cuda_failed(e);
    return h == DEV_OK ? CB_OK : CB_ERR_TIMEOUT;
}

extern "C" cb_status cb_test_hooks(uint32_t poll_limit, int32_t starve_producer)
{
    g_poll_limit.store(poll_limit ? poll_limit : (1u << 22));
    g_starve.store(starve_producer ? 1 : 0);
    return CB_OK;
}

extern "C" int32_t cb_last_cuda_error(const char **text)
{
    const int e = g_last_cuda_error.exchange(0);
    if (text) *text = e ? cudaGetErrorString(static_cast<cudaError_t>(e)) : "no error";
    return e;
}
