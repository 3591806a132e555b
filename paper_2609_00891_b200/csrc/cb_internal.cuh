// Internal declarations shared by the translation units of the library (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "cb.h"

namespace cb {

// ---- partial-statistics slot -------------------------------------------------------------------------
// One slot holds the fp32 partial statistics of one (split, map):
//   D   [d][2d]  D[i][j]     = sum_t w x_i x_j   (j <  d)      -> S_xx
//                D[i][d + j] = sum_t w x_i y_j                 -> S_xy
//   s_x [d], s_y [d], s_w, 3 floats of padding (keeps every slot 16-byte aligned)
__host__ __device__ constexpr int slot_floats(int d) { return d * 2 * d + 2 * d + 4; }
__host__ __device__ constexpr int slot_sx(int d) { return d * 2 * d; }
__host__ __device__ constexpr int slot_sy(int d) { return d * 2 * d + d; }
__host__ __device__ constexpr int slot_sw(int d) { return d * 2 * d + 2 * d; }

// Device-side status word values.
enum : int { DEV_OK = 0, DEV_TIMEOUT = 1 };

// A resolved strided view of K and V (element strides).
struct KVPtr {
    const __nv_bfloat16 *k, *v;
    long long sl, st, sh;
};

struct AccumArgs {
    KVPtr src, tgt;
    const float *w_k, *w_v;
    long long w_sl, w_sh;
    int n_tokens;
    int Lt, Ht, n_splits;
    const int *src_layer;  // device [Lt]
    const int *src_head;   // device [Ht]
    float *slots;          // device [n_splits][n_maps][slot_floats]
    int *status;           // device status word (the context's, else the library's own: library_status_word())
    int compensated;
    unsigned poll_limit = 1u << 22;   // polls after which a bounded device-side wait gives up
    int starve = 0;                   // test hook: the source-tile producer issues nothing, so the waits run out
    // Two-pass centred construction: device [n_maps][2d + 1] = mu_x, mu_y, s_w per map; null for the one-pass path.
    // When set, the weighted operand is w (x - mu_x) and the slot's s_x entries receive the sum of the ROUNDED
    // weighted operand (the exact correction term of the reduction), s_y stays zero.
    const float *mu = nullptr;
    // Rotary embedding at the boundary: device [n_tokens] positions (null: keys are taken as stored) and the rotary
    // bases of the two models.  Key maps are then fitted on de-rotated source and target keys.
    const int *rope_pos = nullptr;
    double rope_base_src = 0.0, rope_base_tgt = 0.0;
};

// First pass of the two-pass construction: fp64 partial sums [n_msplits][n_maps][means_stride(d)] =
// sum w x [d], sum w y [d], sum w, sum w y^2 [d] (the last for the layer selector's total sum of squares), padding.
__host__ __device__ constexpr int means_stride(int d) { return 3 * d + 2; }
constexpr int MEANS_SPLITS = 8;
struct MeansArgs {
    KVPtr src, tgt;
    const float *w_k, *w_v;
    long long w_sl, w_sh;
    int n_tokens;
    int Lt, Ht;
    const int *src_layer;  // device [Lt]
    const int *src_head;   // device [Ht]
    double *msum;          // device [MEANS_SPLITS][n_maps][means_stride(d)]
    // Rotary embedding at the boundary: device [n_tokens] positions (null: keys as stored) and the models' bases; the
    // key maps' sums are then those of the de-rotated rows.
    const int *rope_pos = nullptr;
    double rope_base_src = 0.0, rope_base_tgt = 0.0;
};

struct ApplyArgs {
    KVPtr src;
    const float *Wb;       // [n_maps][p][d]
    void *out_k, *out_v;
    long long o_sl, o_st, o_sh;
    int out_dtype;
    int n_tokens;
    int Lt, Ht;
    int src_layer[128];    // by value: cb_apply takes no context
    int src_head[64];
    // Rotary embedding at the boundary (key maps): device [n_tokens] positions, or null for the ordinary apply.
    const int *rope_pos = nullptr;
    double rope_base_src = 0.0, rope_base_tgt = 0.0;
    int *status = nullptr;            // device status word (the library's own: library_status_word())
    unsigned poll_limit = 1u << 22;   // as in AccumArgs
    int starve = 0;
};

// Full-head contrast statistics: outputs and device tables (see cb_fullhead_stats_accumulate).
struct FullHeadArgs {
    float *G, *C;
    const int *layer_sets, *gi, *gq;   // device
    const int *src_head;               // device [Ht]; used when per_head
    int F, k, Hs, PF, NG, NC, per_head;
};

// Launchers (each returns the cudaError_t of its launch and bumps the launch counter on success).
cudaError_t launch_accum_simt(const AccumArgs &a, int d, cudaStream_t st);
cudaError_t launch_accum_tc(const AccumArgs &a, int d, const cb_kv_view *src, const cb_kv_view *tgt, cudaStream_t st);
cudaError_t launch_accum_ts(const AccumArgs &a, int d, bool comp, const cb_kv_view *src, const cb_kv_view *tgt, cudaStream_t st);
cudaError_t launch_fullhead_tc(const AccumArgs &a, const FullHeadArgs &f, int d, const cb_kv_view *src, const cb_kv_view *tgt,
                               cudaStream_t st);
cudaError_t launch_gram2_tc(const AccumArgs &a, const FullHeadArgs &f, int d, const cb_kv_view *src, const cb_kv_view *tgt,
                            cudaStream_t st);
cudaError_t launch_reduce(const float *slots, int n_splits, int n_maps, int d, float *G, float *C, cudaStream_t st);
cudaError_t launch_means(const MeansArgs &a, int d, cudaStream_t st);
cudaError_t launch_means_finalize(const double *msum, int n_maps, int d, float *mu, cudaStream_t st);
cudaError_t launch_means_energy(const double *msum, int n_maps, int d, float *syy, cudaStream_t st);
cudaError_t launch_probe_r2(const float *G, const float *C, const float *Wb, const float *syy, int n_maps, int d,
                            double lambda, double inv_n, int raw_lambda, float *r2, cudaStream_t st);
cudaError_t launch_probe_scores(const float *r2, int Lt, int Ht, const int *src_layer_host, int Ls, float *scores, cudaStream_t st);
cudaError_t launch_reduce_centered(const float *slots, int n_splits, int n_maps, int d, const float *mu, float *A, float *B,
                                   int k_operands_centred, cudaStream_t st);
cudaError_t launch_solve_centered(const float *A, const float *B, const float *mu, int n_maps, int d, long long n_tokens,
                                  const float *lambdas, int n_lambda, unsigned flags, float *Wb, int *info, cudaStream_t st);
cudaError_t launch_solve(const float *G, const float *C, int n_maps, int d, long long n_tokens,
                         const float *lambdas, int n_lambda, unsigned flags, float *Wb, int *info, cudaStream_t st);
size_t solve_large_bytes_per_system(int P, int d);
cudaError_t launch_solve_large(const float *G, const float *C, int n_maps, int P, int d, long long n_tokens,
                               const float *lambdas, int n_lambda, unsigned flags, float *Wb, int *info,
                               void *workspace, size_t workspace_bytes, cudaStream_t st);
cudaError_t launch_apply_simt(const ApplyArgs &a, int d, cudaStream_t st);
cudaError_t launch_apply_tc(const ApplyArgs &a, int d, const cb_kv_view *src, cudaStream_t st);

size_t apply_ml_workspace_bytes(int n_maps, int k, int d, int Lt);
cudaError_t launch_apply_ml_tc(const ApplyArgs &a, int d, int k, const int *layer_sets_host, const cb_kv_view *src,
                               void *workspace, cudaStream_t st);

cudaError_t launch_rope_rotate(void *k, int L, int H, int d, long long T, long long sl, long long st, long long sh,
                               const int *pos, double base, int inverse, cudaStream_t stream);

void count_launch(int n = 1);

// 5-D tensor map over (64 channels, token, 64-channel block, head, layer) of a strided bf16 K or V tensor.  One box =
// box_tokens tokens of one head of one layer, laid out in shared memory as [channel block][token][64 channels] with
// the 128-byte swizzle; box_cblocks = 64-channel blocks per box (0: all d / 64 of them; 1: one block, selected by the
// copy's third coordinate).
bool make_kv_tensor_map(CUtensorMap *map, const void *base, int d, int H, long long T, int L,
                        long long sh, long long st, long long sl, int box_tokens, int box_cblocks = 0);

// Host-side argument checks shared by the entry points (status codes of the C ABI).
cb_status check_problem(const cb_problem *p);
cb_status check_view(const cb_kv_view *v, int L, int H, int d);

// ---- per-device host state ---------------------------------------------------------------------------
constexpr int MAX_DEVICES = 64;
// SM count of the current device (asked once per device; 148 if there is no device to ask).
int device_sm_count();
// Device address, on the current device, of the library's own status word: kernels launched without a context
// record a device-side time-out there and cb_last_device_status reads it.  Null if the lookup failed.
int *library_status_word();
// A CUDA runtime call failed: remembers its error code for cb_last_cuda_error (`e`, or the runtime's last error when
// the caller has none), clears the runtime's last-error state and returns CB_ERR_CUDA.
cb_status cuda_failed(cudaError_t e = cudaSuccess);

// Test hooks (cb_test_hooks): poll limit of the bounded waits and the starved-producer switch for later launches.
struct TestHooks { unsigned poll_limit; int starve; };
TestHooks test_hooks();
// Opt a kernel in to more than 48 KB of dynamic shared memory, once per device.
template <class K>
inline cudaError_t opt_in_smem(K kernel, size_t bytes, bool (&done)[MAX_DEVICES])
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    if (!done[dev]) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        if (e != cudaSuccess) return e;
        done[dev] = true;
    }
    return cudaSuccess;
}

}  // namespace cb
