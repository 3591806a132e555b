// Fused weighted-statistics accumulation on the 5th-generation tensor cores (sm_100a).
//
// For one map (matched source head X, target head Y, token weights w) the statistics are the dense contraction
//     D[d][2d] = (w .* X)^T [X | Y]          over tokens,
// plus the bias sums s_x = sum w x, s_y = sum w y, s_w = sum w kept on the ALUs.
//
// Per thread block (one per SM, persistent over its units = (map, token split)):
//   warp 0      TMA producer: tiles of TT tokens of X and Y go straight from the strided cache layout to shared
//               memory (128-byte swizzle: one row = one token's 64 channels), NS stages deep.
//   warps 2-9   fold: read the X tile, multiply each token row by its weight, round to bf16 (optionally hi+lo)
//               into the A buffer in the same swizzled layout; accumulate the bias sums in registers.
//   warp 1      MMA issuer: tcgen05.mma, A = weighted tile (M = 128 channels, MN-major), B = [X | Y]
//               (N = 2d channels, MN-major), K = tokens, fp32 accumulator in tensor memory.
//   warps 10-13 drain: when a unit's accumulator is complete, tensor memory -> registers -> read-modify-write of
//               the unit's fp32 partial slot; two accumulators let the next unit start meanwhile.
// Every wait is bounded: if one runs out the block sets the context's status word and tears down.
#include <cudaTypedefs.h>

#include "cb_internal.cuh"
#include "cb_ptx.cuh"

namespace cb {

using namespace ptx;

template <int D>
struct TcCfg {
    static constexpr int TT = 64;                     // tokens per tile
    static constexpr int NBX = D / 64;                // 64-channel blocks per head
    static constexpr int BLK = TT * 128;              // bytes of one block: TT rows of 128 bytes
    static constexpr int STAGE_BYTES = 2 * NBX * BLK; // X blocks, then Y blocks
    static constexpr int A_BYTES = 2 * BLK;           // M = 128 always: two blocks (second stays zero for d = 64)
    static constexpr int NS = 4;                      // X/Y stages
    static constexpr int NA = 2;                      // weighted-operand buffers (each hi + lo)
    static constexpr int N = 2 * D;                   // accumulator columns
    static constexpr int TMEM_COLS = 2 * N;           // two accumulators
    static constexpr int FOLD_WARPS = 8, DRAIN_WARPS = 4;
    static constexpr int FOLD_THREADS = FOLD_WARPS * 32;
    static constexpr int THREADS = (2 + FOLD_WARPS + DRAIN_WARPS) * 32;
    static constexpr int CC = D / 8;                  // 16-byte chunk columns of a head row
    static constexpr int RG = FOLD_THREADS / CC;      // row groups
    static constexpr int RPT = TT / RG;               // rows per fold thread
    static constexpr int RED_STRIDE = 2 * D + 4;                 // per fold warp: s_x[D], s_y[D], s_w, pad
    static constexpr int RED_FLOATS = FOLD_WARPS * RED_STRIDE;      // cross-warp bias reduction buffer
    static constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)NS * STAGE_BYTES + (size_t)NA * 2 * A_BYTES +
                                         RED_FLOATS * 4 + 256 /*barriers*/;
    static_assert(TT % RG == 0 && RPT >= 1, "fold layout");
    static_assert(TMEM_COLS == 256 || TMEM_COLS == 512, "tensor memory columns must be a power of two");
};

struct TcParams {
    CUtensorMap src_k, src_v, tgt_k, tgt_v;   // 4-D tiled maps, innermost dimension = channels
    AccumArgs a;
    int s_pos[3], t_pos[3];                   // coordinate slot (1..3) of head, token, layer in each map
    int drain_tiles;                          // tiles accumulated in tensor memory between drains
};

__device__ __forceinline__ void unpack_bf16x8(const uint4 &v, float *f)
{
    const unsigned u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(u[i] << 16);
        f[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi)
{
    unsigned r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

template <int D>
__global__ void __launch_bounds__(TcCfg<D>::THREADS, 1) k_accum_tc(const __grid_constant__ TcParams P)
{
    using C = TcCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *xy = smem;                                       // [NS][STAGE_BYTES]
    uint8_t *ab = xy + (size_t)C::NS * C::STAGE_BYTES;        // [NA][hi A_BYTES | lo A_BYTES]
    float *red = reinterpret_cast<float *>(ab + (size_t)C::NA * 2 * C::A_BYTES);
    uint64_t *bars = reinterpret_cast<uint64_t *>(red + C::RED_FLOATS);
    uint64_t *full = bars;                 // [NS] TMA landed
    uint64_t *empty = full + C::NS;        // [NS] stage free: MMA done (1) + fold warps done (8)
    uint64_t *afull = empty + C::NS;       // [NA] weighted operand written (8 fold warps)
    uint64_t *aempty = afull + C::NA;      // [NA] weighted operand consumed (MMA)
    uint64_t *accfull = aempty + C::NA;    // [2]  accumulator complete (MMA)
    uint64_t *accempty = accfull + 2;      // [2]  accumulator drained (4 drain warps)
    uint64_t *redfull = accempty + 2;      // [1]  bias partials of all fold warps written
    uint64_t *reddone = redfull + 1;       // [1]  bias partials consumed
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(reddone + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const AccumArgs &a = P.a;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_maps = 2 * a.Lt * a.Ht;
    const int n_units = n_maps * a.n_splits;
    const int n_tiles = (a.n_tokens + C::TT - 1) / C::TT;

    if (tid == 0) {
        for (int i = 0; i < C::NS; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1 + C::FOLD_WARPS); }
        for (int i = 0; i < C::NA; ++i) { mbar_init(&afull[i], C::FOLD_WARPS); mbar_init(&aempty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&accfull[i], 1); mbar_init(&accempty[i], C::DRAIN_WARPS); }
        mbar_init(redfull, C::FOLD_WARPS);
        mbar_init(reddone, C::FOLD_WARPS);
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&P.src_k); tma_prefetch_desc(&P.src_v);
        tma_prefetch_desc(&P.tgt_k); tma_prefetch_desc(&P.tgt_v);
    }
    if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
    if (D == 64 && warp >= 2 && warp < 2 + C::FOLD_WARPS) {
        // rows 64..127 of the M = 128 operand never get data: clear the second block of every A buffer once
        const int ft = tid - 64;
        for (int i = ft; i < C::NA * 2 * (C::BLK / 16); i += C::FOLD_THREADS) {
            const int buf = i / (C::BLK / 16), off = i % (C::BLK / 16);
            *reinterpret_cast<uint4 *>(ab + (size_t)buf * C::A_BYTES + C::BLK + off * 16) = make_uint4(0, 0, 0, 0);
        }
        fence_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Every role walks the same sequence: units u = blockIdx.x, += gridDim.x; unit -> (map, split) -> tiles
    // [tile0, tile1); sub-ranges of at most drain_tiles tiles share one accumulator.
    if (warp == 0) {
        // ================================ TMA producer ================================
        if (lane == 0) {
            uint32_t it = 0;
            for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
                const int m = u % n_maps, split = u / n_maps;
                const int tile0 = (int)(((long long)n_tiles * split) / a.n_splits);
                const int tile1 = (int)(((long long)n_tiles * (split + 1)) / a.n_splits);
                const int comp = m / (a.Lt * a.Ht), l = (m / a.Ht) % a.Lt, h = m % a.Ht;
                const int j = a.src_layer[l], g = a.src_head[h];
                const CUtensorMap *ms = comp ? &P.src_v : &P.src_k;
                const CUtensorMap *mt = comp ? &P.tgt_v : &P.tgt_k;
                for (int tile = tile0; tile < tile1; ++tile, ++it) {
                    const int s = it % C::NS;
                    if (!mbar_wait(&empty[s], ((it / C::NS) & 1) ^ 1, abort_flag)) goto teardown;
                    mbar_arrive_expect_tx(&full[s], C::STAGE_BYTES);
                    uint8_t *dst = xy + (size_t)s * C::STAGE_BYTES;
                    int cs[4], ct[4];
                    cs[P.s_pos[0]] = g; cs[P.s_pos[1]] = tile * C::TT; cs[P.s_pos[2]] = j;
                    ct[P.t_pos[0]] = h; ct[P.t_pos[1]] = tile * C::TT; ct[P.t_pos[2]] = l;
#pragma unroll
                    for (int b = 0; b < C::NBX; ++b) {
                        tma_load_4d(dst + b * C::BLK, ms, &full[s], b * 64, cs[1], cs[2], cs[3]);
                        tma_load_4d(dst + (C::NBX + b) * C::BLK, mt, &full[s], b * 64, ct[1], ct[2], ct[3]);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ================================ MMA issuer ================================
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, C::N, true, true);
            uint32_t it = 0, sr = 0;
            for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
                const int split = u / n_maps;
                const int tile0 = (int)(((long long)n_tiles * split) / a.n_splits);
                const int tile1 = (int)(((long long)n_tiles * (split + 1)) / a.n_splits);
                for (int sr0 = tile0; sr0 < tile1; sr0 += P.drain_tiles, ++sr) {
                    const int sr1 = min(tile1, sr0 + P.drain_tiles);
                    const int acc = sr & 1;
                    if (!mbar_wait(&accempty[acc], ((sr >> 1) & 1) ^ 1, abort_flag)) goto teardown;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * C::N;
                    for (int tile = sr0; tile < sr1; ++tile, ++it) {
                        const int s = it % C::NS, ai = it % C::NA;
                        if (!mbar_wait(&full[s], (it / C::NS) & 1, abort_flag)) goto teardown;
                        if (!mbar_wait(&afull[ai], (it / C::NA) & 1, abort_flag)) goto teardown;
                        tc_fence_after();
                        const uint32_t b_addr = smem_u32(xy + (size_t)s * C::STAGE_BYTES);
                        const uint32_t a_addr = smem_u32(ab + (size_t)ai * 2 * C::A_BYTES);
#pragma unroll
                        for (int k = 0; k < C::TT / 16; ++k) {
                            const uint64_t bd = umma_smem_desc_sw128(b_addr + k * 2048, C::BLK, 1024);
                            const uint64_t ad = umma_smem_desc_sw128(a_addr + k * 2048, C::BLK, 1024);
                            umma_bf16_ss(d_tmem, ad, bd, idesc, (tile > sr0 || k > 0) ? 1u : 0u);
                            if (a.compensated) {
                                const uint64_t ld = umma_smem_desc_sw128(a_addr + C::A_BYTES + k * 2048, C::BLK, 1024);
                                umma_bf16_ss(d_tmem, ld, bd, idesc, 1u);
                            }
                        }
                        umma_commit(&empty[s]);
                        umma_commit(&aempty[ai]);
                    }
                    umma_commit(&accfull[acc]);
                }
            }
        }
    } else if (warp < 2 + C::FOLD_WARPS) {
        // ================================ fold warps ================================
        const int ft = tid - 64;
        const int cc = ft % C::CC, rg = ft / C::CC;
        const int blk = cc >> 3, lc = cc & 7;
        float sx[8], sy[8], sw = 0.f;
        uint32_t it = 0, uc = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            const int m = u % n_maps, split = u / n_maps;
            const int tile0 = (int)(((long long)n_tiles * split) / a.n_splits);
            const int tile1 = (int)(((long long)n_tiles * (split + 1)) / a.n_splits);
            if (tile0 >= tile1) continue;
            const int comp = m / (a.Lt * a.Ht), l = (m / a.Ht) % a.Lt, h = m % a.Ht;
            const float *w = (comp ? a.w_v : a.w_k) + (long long)l * a.w_sl + (long long)h * a.w_sh;
#pragma unroll
            for (int e = 0; e < 8; ++e) sx[e] = sy[e] = 0.f;
            sw = 0.f;
            float wn[C::RPT];
#pragma unroll
            for (int i = 0; i < C::RPT; ++i) {
                const int t = tile0 * C::TT + rg + i * C::RG;
                wn[i] = (t < a.n_tokens) ? __ldg(w + t) : 0.f;
            }
            for (int tile = tile0; tile < tile1; ++tile, ++it) {
                float wc[C::RPT];
#pragma unroll
                for (int i = 0; i < C::RPT; ++i) wc[i] = wn[i];
                if (tile + 1 < tile1) {
#pragma unroll
                    for (int i = 0; i < C::RPT; ++i) {
                        const int t = (tile + 1) * C::TT + rg + i * C::RG;
                        wn[i] = (t < a.n_tokens) ? __ldg(w + t) : 0.f;
                    }
                }
                const int s = it % C::NS, ai = it % C::NA;
                {
                    bool ok = mbar_wait(&full[s], (it / C::NS) & 1, abort_flag);
                    ok = ok && mbar_wait(&aempty[ai], ((it / C::NA) & 1) ^ 1, abort_flag);
                    if (!__all_sync(0xffffffffu, ok)) goto teardown;
                }
                const uint8_t *xs = xy + (size_t)s * C::STAGE_BYTES + blk * C::BLK;
                const uint8_t *ys = xs + C::NBX * C::BLK;
                uint8_t *ah = ab + (size_t)ai * 2 * C::A_BYTES + blk * C::BLK;
#pragma unroll
                for (int i = 0; i < C::RPT; ++i) {
                    const int r = rg + i * C::RG;
                    const int off = r * 128 + ((lc ^ (r & 7)) << 4);
                    const float wt = wc[i];
                    float f[8], pr[8];
                    unpack_bf16x8(*reinterpret_cast<const uint4 *>(xs + off), f);
#pragma unroll
                    for (int e = 0; e < 8; ++e) { pr[e] = wt * f[e]; sx[e] += pr[e]; }
                    uint4 hi;
                    hi.x = pack_bf16x2(pr[0], pr[1]); hi.y = pack_bf16x2(pr[2], pr[3]);
                    hi.z = pack_bf16x2(pr[4], pr[5]); hi.w = pack_bf16x2(pr[6], pr[7]);
                    *reinterpret_cast<uint4 *>(ah + off) = hi;
                    if (a.compensated) {
                        float hf[8];
                        unpack_bf16x8(hi, hf);
                        uint4 lo;
                        lo.x = pack_bf16x2(pr[0] - hf[0], pr[1] - hf[1]); lo.y = pack_bf16x2(pr[2] - hf[2], pr[3] - hf[3]);
                        lo.z = pack_bf16x2(pr[4] - hf[4], pr[5] - hf[5]); lo.w = pack_bf16x2(pr[6] - hf[6], pr[7] - hf[7]);
                        *reinterpret_cast<uint4 *>(ah + C::A_BYTES + off) = lo;
                    }
                    unpack_bf16x8(*reinterpret_cast<const uint4 *>(ys + off), f);
#pragma unroll
                    for (int e = 0; e < 8; ++e) sy[e] = fmaf(wt, f[e], sy[e]);
                    if (cc == 0) sw += wt;
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&afull[ai]); mbar_arrive(&empty[s]); }
            }
            // ---- bias sums of this unit: lanes pair up (two row groups per warp when CC = 16), then a fixed-order
            //      sum over the warps, then read-modify-write of the slot ----
            if (C::CC == 16) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    sx[e] += __shfl_xor_sync(0xffffffffu, sx[e], 16);
                    sy[e] += __shfl_xor_sync(0xffffffffu, sy[e], 16);
                }
                sw += __shfl_xor_sync(0xffffffffu, sw, 16);
            } else {   // CC = 8: four row groups per warp
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    sx[e] += __shfl_xor_sync(0xffffffffu, sx[e], 8);
                    sy[e] += __shfl_xor_sync(0xffffffffu, sy[e], 8);
                    sx[e] += __shfl_xor_sync(0xffffffffu, sx[e], 16);
                    sy[e] += __shfl_xor_sync(0xffffffffu, sy[e], 16);
                }
                sw += __shfl_xor_sync(0xffffffffu, sw, 8);
                sw += __shfl_xor_sync(0xffffffffu, sw, 16);
            }
            const int fw = warp - 2;
            // red[fw][v], v in [0, 2D): s_x channels then s_y channels; red[fw][2D] = s_w
            if (!__all_sync(0xffffffffu, mbar_wait(reddone, (uc & 1) ^ 1, abort_flag))) goto teardown;
            float *rw = red + fw * C::RED_STRIDE;
            if (lane < C::CC) {
#pragma unroll
                for (int e = 0; e < 8; ++e) { rw[cc * 8 + e] = sx[e]; rw[D + cc * 8 + e] = sy[e]; }
                if (cc == 0) rw[2 * D] = sw;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(redfull);
            if (!__all_sync(0xffffffffu, mbar_wait(redfull, uc & 1, abort_flag))) goto teardown;
            float *slot = a.slots + ((size_t)split * n_maps + m) * slot_floats(D);
            for (int v = ft; v < 2 * D + 1; v += C::FOLD_THREADS) {
                float sum = 0.f;
#pragma unroll
                for (int q = 0; q < C::FOLD_WARPS; ++q) sum += red[q * C::RED_STRIDE + v];
                slot[slot_sx(D) + v] += sum;    // s_x, s_y, s_w are adjacent in the slot
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(reddone);
            ++uc;
        }
    } else {
        // ================================ drain warps ================================
        const int q = warp & 3;             // tensor-memory lane quarter this warp may access
        const int row = q * 32 + lane;      // row of D = channel of the weighted operand
        uint32_t sr = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            const int m = u % n_maps, split = u / n_maps;
            const int tile0 = (int)(((long long)n_tiles * split) / a.n_splits);
            const int tile1 = (int)(((long long)n_tiles * (split + 1)) / a.n_splits);
            float *slot = a.slots + ((size_t)split * n_maps + m) * slot_floats(D);
            for (int sr0 = tile0; sr0 < tile1; sr0 += P.drain_tiles, ++sr) {
                const int acc = sr & 1;
                if (!__all_sync(0xffffffffu, mbar_wait(&accfull[acc], (sr >> 1) & 1, abort_flag))) goto teardown;
                tc_fence_after();
                if (row < D) {
                    float *grow = slot + (size_t)row * C::N;
#pragma unroll 1
                    for (int c = 0; c < C::N / 32; ++c) {
                        uint32_t r[32];
                        float4 g[8];
#pragma unroll
                        for (int v = 0; v < 8; ++v) g[v] = *reinterpret_cast<const float4 *>(grow + c * 32 + v * 4);
                        tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + acc * C::N + c * 32, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            g[v].x += __uint_as_float(r[4 * v + 0]);
                            g[v].y += __uint_as_float(r[4 * v + 1]);
                            g[v].z += __uint_as_float(r[4 * v + 2]);
                            g[v].w += __uint_as_float(r[4 * v + 3]);
                            *reinterpret_cast<float4 *>(grow + c * 32 + v * 4) = g[v];
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&accempty[acc]);
            }
        }
    }

teardown:
    __syncwarp();
    if (*abort_flag) {
        if (tid == 0) atomicExch(a.status, DEV_TIMEOUT);
        // give copies that may still be in flight time to land before the block's shared memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------------
// Host: tensor maps and launch
// ------------------------------------------------------------------------------------------------------
static PFN_cuTensorMapEncodeTiled_v12000 encode_fn()
{
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
    }
    return fn;
}

// 4-D map over (channels, and head/token/layer ordered by ascending stride); pos[0..2] receive the coordinate
// slot of head, token and layer.  Box: 64 channels x box_tokens tokens of one head of one layer.
bool make_kv_tensor_map(CUtensorMap *map, const void *base, int d, int H, long long T, int L,
                        long long sh, long long st, long long sl, int box_tokens, int pos[3])
{
    PFN_cuTensorMapEncodeTiled_v12000 enc = encode_fn();
    if (!enc) return false;
    struct Dim { unsigned long long size, stride_bytes; int which; };
    Dim dims[3] = {{(unsigned long long)H, (unsigned long long)sh * 2, 0},
                   {(unsigned long long)T, (unsigned long long)st * 2, 1},
                   {(unsigned long long)L, (unsigned long long)sl * 2, 2}};
    for (int i = 0; i < 3; ++i)
        if (dims[i].size == 1 || dims[i].stride_bytes == 0) dims[i].stride_bytes = 0;   // placed first, fixed below
    // ascending stride (stable insertion sort)
    for (int i = 1; i < 3; ++i)
        for (int k = i; k > 0 && dims[k].stride_bytes < dims[k - 1].stride_bytes; --k) { Dim t = dims[k]; dims[k] = dims[k - 1]; dims[k - 1] = t; }
    cuuint64_t gdim[4] = {(cuuint64_t)d, 1, 1, 1};
    cuuint64_t gstr[3];
    cuuint32_t box[4] = {64, 1, 1, 1}, estr[4] = {1, 1, 1, 1};
    for (int i = 0; i < 3; ++i) {
        gdim[i + 1] = dims[i].size;
        unsigned long long sb = dims[i].stride_bytes;
        if (sb == 0) sb = (unsigned long long)d * 2;   // size-1 dimension: any valid stride
        gstr[i] = sb;
        pos[dims[i].which] = i + 1;
        if (dims[i].which == 1) box[i + 1] = (cuuint32_t)box_tokens;
    }
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), gdim, gstr, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

static int sm_count()
{
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

template <int D>
static cudaError_t launch_tc(const TcParams &P, cudaStream_t st)
{
    using C = TcCfg<D>;
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(k_accum_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    const int n_units = 2 * P.a.Lt * P.a.Ht * P.a.n_splits;
    const int grid = n_units < sm_count() ? n_units : sm_count();
    k_accum_tc<D><<<grid, C::THREADS, C::SMEM_BYTES, st>>>(P);
    return cudaGetLastError();
}

cudaError_t launch_accum_tc(const AccumArgs &a, int d, const cb_kv_view *src, const cb_kv_view *tgt, cudaStream_t st)
{
    TcParams P;
    P.a = a;
    const int TT = 64;
    if (!make_kv_tensor_map(&P.src_k, src->k, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                            src->stride_token, src->stride_layer, TT, P.s_pos) ||
        !make_kv_tensor_map(&P.src_v, src->v, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                            src->stride_token, src->stride_layer, TT, P.s_pos) ||
        !make_kv_tensor_map(&P.tgt_k, tgt->k, d, tgt->n_heads, tgt->n_tokens, tgt->n_layers, tgt->stride_head,
                            tgt->stride_token, tgt->stride_layer, TT, P.t_pos) ||
        !make_kv_tensor_map(&P.tgt_v, tgt->v, d, tgt->n_heads, tgt->n_tokens, tgt->n_layers, tgt->stride_head,
                            tgt->stride_token, tgt->stride_layer, TT, P.t_pos))
        return cudaErrorInvalidValue;
    P.drain_tiles = 16384 / TT;   // at most 16384 tokens are summed in tensor memory before a drain
    cudaError_t e = (d == 128) ? launch_tc<128>(P, st) : launch_tc<64>(P, st);
    if (e == cudaSuccess) count_launch();
    return e;
}

}  // namespace cb
