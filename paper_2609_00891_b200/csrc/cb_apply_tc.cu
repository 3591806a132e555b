// Online affine apply on the tensor cores (sm_100a):  out[t][:] = x_t W + b  for every map and token.
//
// Per thread block (persistent; units = (map, token range)):
//   conversion warps  split the map's fp32 W into bf16 hi + lo and write both into shared memory in the layout the
//                     tensor core reads (rows = input channel, 64 output channels per 128-byte row, swizzled);
//                     the bias row goes to shared memory as fp32.
//   producer thread   TMA: tiles of 128 tokens of the matched source head, [channel block][token][64 channels].
//   MMA thread        tcgen05.mma  D[128 tokens][d] += X[128][16] * W_hi[16][d], then the same with W_lo, A K-major,
//                     B MN-major: both products accumulate into the same tensor-memory columns, so the epilogue has
//                     no halves to add (one N = 2d operand with the halves added in registers measured 1.5 % slower:
//                     like the statistics kernel, this one is limited by the board's power, and 128 fp32 adds per
//                     row cost more than a second read of the X tile by the tensor cores); four fp32 accumulators
//                     in tensor memory.
//   epilogue warps    tensor memory -> registers, + bias, -> bf16 into a shared-memory tile -> one TMA store
//                     (coalesced 256-byte rows, rows past the end clipped); fp32 output is stored directly.
// Every wait is bounded; a wait that runs out makes the block set the library's status word (cb_last_device_status)
// and tear down.
#include <cudaTypedefs.h>

#include <cuda_fp16.h>

#include <algorithm>
#include <vector>

#include "cb_internal.cuh"
#include "cb_ptx.cuh"
#include "cb_math.cuh"
#include "cb_rope.cuh"

namespace cb {

using namespace ptx;

// Rotary kernels: eight epilogue warps (two sets of four, a set takes every other column group of a tile).  Measured on
// the 32,768-token cache of the 14B -> 32B shapes, interleaved runs: 4 epilogue + 4 conversion warps 4.00 ms, 8 + 4
// 3.79 ms, 4 + 8 4.80 ms, 8 + 8 4.02 ms (more conversion threads means shorter row blocks, so more first rows that
// need the special-function unit); sending 4 or 8 of every 16 epilogue angles through the FMA-pipe polynomial
// instead of the special-function unit: 4.0 / 4.4 ms.  With the epilogue's angles or the source rotation left out the
// time falls by 0.3 - 0.5 ms each, with both left out to 3.0 ms (2.77 ms without the rotary boundary): the key maps'
// tiles are bound by the sum of the two roles' instructions, not by one of them.
constexpr int ROPE_EPI_WARPS = 8;

template <int D, int EW = 4>
struct ApCfg {
    static constexpr int TT = 128;                      // tokens per tile = MMA M
    static constexpr int NB = D / 64;                   // 64-channel blocks
    static constexpr int XBLK = TT * 128;               // bytes of one X block
    static constexpr int X_BYTES = NB * XBLK;           // one X stage
    static constexpr int WBLK = D * 128;                // bytes of one W block: D rows (input channels) of 128 bytes
    static constexpr int W_BYTES = NB * WBLK;           // hi (or lo) part of W
    static constexpr int O_BYTES = NB * XBLK;           // bf16 output tile
    static constexpr int NS = 3;
    static constexpr int NO = 2;                 // output tiles in shared memory
    static constexpr int NACC = 4;
    static constexpr int AW = D;                        // accumulator columns per tile: X W_hi + X W_lo
    static constexpr int TMEM_COLS = (NACC * AW < 32) ? 32 : NACC * AW;
    static constexpr int EPI_WARPS = EW, CONV_WARPS = 4;  // EW = 8: two sets of four, each takes every other column group
    static constexpr int THREADS = (2 + EPI_WARPS + CONV_WARPS) * 32;
    static constexpr size_t SMEM_BYTES = 1024 + (size_t)NS * X_BYTES + 2 * (size_t)W_BYTES + (size_t)NO * O_BYTES + D * 4 + 256;
};

struct ApParams {
    CUtensorMap src_k, src_v, out_k, out_v;
    ApplyArgs a;
    int n_splits;
    RopeDev rope;        // ROPE kernels only
};

struct ApIter {   // units u = blockIdx.x, += gridDim.x; unit -> (map, split) -> tiles [tile, tile1)
    int u, tile, tile1, m;
    __device__ __forceinline__ void next_unit(int n_units, int n_maps, int n_tiles, int n_splits)
    {
        do {
            u += gridDim.x;
            if (u >= n_units) return;
            m = u % n_maps;
            const int split = u / n_maps;
            tile = (int)(((long long)n_tiles * split) / n_splits);
            tile1 = (int)(((long long)n_tiles * (split + 1)) / n_splits);
        } while (tile >= tile1);
    }
    __device__ __forceinline__ void start(int n_units, int n_maps, int n_tiles, int n_splits)
    {
        u = (int)blockIdx.x - (int)gridDim.x;
        tile = tile1 = 0;
        next_unit(n_units, n_maps, n_tiles, n_splits);
    }
};

// fp16 pair (low half = first element)
__device__ __forceinline__ unsigned ap_pack_f16x2(float lo, float hi)
{
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const unsigned *>(&h);
}

// ROPE (Section 3.1: source RoPE removed before the map, target RoPE restored after it): for key maps (comp = 0) the
// conversion warps rotate every staged source tile back by its rows' angles in place, writing fp16 (the rotated
// values are no longer bf16 numbers: fp16 keeps 11 significant bits, and W is split into fp16 hi + lo to match), the
// tensor cores run with fp16 operands, and the epilogue rotates the mapped rows forward by the target model's angles.
// Value maps take the ordinary bf16 path through the same barriers.
template <int D, bool ROPE>
__global__ void __launch_bounds__(ApCfg<D, ROPE ? ROPE_EPI_WARPS : 4>::THREADS, 1) k_apply_tc(const __grid_constant__ ApParams P)
{
    using C = ApCfg<D, ROPE ? ROPE_EPI_WARPS : 4>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *xs = smem;                                   // [NS][X_BYTES]
    uint8_t *whi = xs + (size_t)C::NS * C::X_BYTES;       // [NB][D rows][128 B]
    uint8_t *wlo = whi + C::W_BYTES;
    uint8_t *os = wlo + C::W_BYTES;                       // [NB][TT rows][128 B] bf16 output tile
    float *bias = reinterpret_cast<float *>(os + (size_t)C::NO * C::O_BYTES);
    uint64_t *bars = reinterpret_cast<uint64_t *>(bias + D);
    uint64_t *xfull = bars;                  // [NS]
    uint64_t *xempty = xfull + C::NS;        // [NS]   MMA done with the stage
    uint64_t *accfull = xempty + C::NS;      // [NACC] accumulator complete
    uint64_t *accempty = accfull + C::NACC;  // [NACC] accumulator read out (EPI_WARPS arrivals)
    uint64_t *wready = accempty + C::NACC;   // [1]    W of the current unit converted (CONV_WARPS arrivals)
    uint64_t *wfree = wready + 1;            // [1]    last MMA of the unit done: W may be overwritten
    uint64_t *bfree = wfree + 1;             // [1]    bias of the unit no longer needed (EPI_WARPS arrivals)
    uint64_t *owritten = bfree + 1;          // [NO]   output tile written by all epilogue warps
    uint64_t *ofree = owritten + C::NO;      // [NO]   output tile read by its store
    uint64_t *xrot = ofree + C::NO;          // [NS]   ROPE: source tile ready for the tensor cores (CONV_WARPS arrivals)
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(xrot + C::NS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const ApplyArgs &a = P.a;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_maps = 2 * a.Lt * a.Ht;
    const int n_units = n_maps * P.n_splits;
    const int n_tiles = (a.n_tokens + C::TT - 1) / C::TT;
    const bool out_bf16 = a.out_dtype == CB_DTYPE_BF16;

    if (tid == 0) {
        for (int i = 0; i < C::NS; ++i) { mbar_init(&xfull[i], 1); mbar_init(&xempty[i], 1); mbar_init(&xrot[i], C::CONV_WARPS); }
        for (int i = 0; i < C::NACC; ++i) { mbar_init(&accfull[i], 1); mbar_init(&accempty[i], C::EPI_WARPS); }
        mbar_init(wready, C::CONV_WARPS);
        mbar_init(wfree, 1);
        mbar_init(bfree, C::EPI_WARPS);
        for (int i = 0; i < C::NO; ++i) { mbar_init(&owritten[i], C::EPI_WARPS); mbar_init(&ofree[i], 1); }
        abort_flag[0] = 0;
        abort_flag[1] = (int)P.a.poll_limit;
        mbar_fence_init();
        tma_prefetch_desc(&P.src_k); tma_prefetch_desc(&P.src_v);
        tma_prefetch_desc(&P.out_k); tma_prefetch_desc(&P.out_v);
    }
    if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ================================ producer (one thread) ================================
        if (lane == 0 && !a.starve) {       // starve (test hook): no source tile is ever requested
            ApIter cur;
            cur.start(n_units, n_maps, n_tiles, P.n_splits);
            Ring<C::NS> st;
            while (cur.u < n_units) {
                const int m = cur.m;
                const int comp = m / (a.Lt * a.Ht), l = (m / a.Ht) % a.Lt, h = m % a.Ht;
                const CUtensorMap *map = comp ? &P.src_v : &P.src_k;
                const int j = a.src_layer[l], g = a.src_head[h];
                for (int tile = cur.tile; tile < cur.tile1; ++tile) {
                    if (!mbar_wait(&xempty[st.idx], st.phase ^ 1, abort_flag)) goto teardown;
                    mbar_arrive_expect_tx(&xfull[st.idx], C::X_BYTES);
                    tma_load_5d(xs + st.idx * C::X_BYTES, map, &xfull[st.idx], 0, tile * C::TT, 0, g, j);
                    st.next();
                }
                cur.next_unit(n_units, n_maps, n_tiles, P.n_splits);
            }
        }
    } else if (warp == 1) {
        // ================================ MMA issuer (one thread) ================================
        if (lane == 0) {
            constexpr uint32_t idesc_bf = umma_idesc_bf16(128, C::AW, false, true);   // A K-major, B MN-major
            constexpr uint32_t idesc_hf = umma_idesc_f16(128, C::AW, false, true);
            // A (K-major, 128-byte swizzle): 8-row groups 1024 bytes apart; a K step of 16 channels is 32 bytes along
            // the row, a block of 64 channels is XBLK further.  B (MN-major): K step = 16 rows = 2048 bytes,
            // 64-output-channel blocks WBLK apart.
            const uint64_t proto_a = umma_smem_desc_sw128(0, 16, 1024);
            const uint64_t proto_b = umma_smem_desc_sw128(0, C::WBLK, 1024);
            const uint32_t a_hi32 = (uint32_t)(proto_a >> 32), b_hi32 = (uint32_t)(proto_b >> 32);
            const uint32_t a_lo0 = (uint32_t)proto_a | ((smem_u32(xs) & 0x3FFFFu) >> 4);
            const uint32_t bh_lo0 = (uint32_t)proto_b | ((smem_u32(whi) & 0x3FFFFu) >> 4);
            ApIter cur;
            cur.start(n_units, n_maps, n_tiles, P.n_splits);
            Ring<C::NS> st;
            Ring<C::NACC> ac;
            uint32_t uc = 0;
            while (cur.u < n_units) {
                if (!mbar_wait(wready, uc & 1, abort_flag)) goto teardown;
                const uint32_t idesc = (ROPE && cur.m < a.Lt * a.Ht) ? idesc_hf : idesc_bf;   // key maps of a ROPE launch: fp16
                for (int tile = cur.tile; tile < cur.tile1; ++tile) {
                    // ROPE launches: every tile passes through the conversion warps (which rotate key tiles)
                    if (!mbar_wait(ROPE ? &xrot[st.idx] : &xfull[st.idx], st.phase, abort_flag)) goto teardown;
                    if (!mbar_wait(&accempty[ac.idx], ac.phase ^ 1, abort_flag)) goto teardown;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + ac.idx * C::AW;
                    const uint32_t al = a_lo0 + st.idx * (C::X_BYTES >> 4);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t ak = al + (k >> 2) * (C::XBLK >> 4) + (k & 3) * 2;          // +32 bytes per K step
                        const uint64_t ad = ((uint64_t)a_hi32 << 32) | ak;
                        // the lo image follows the hi image in shared memory: 2 d / 64 column blocks, WBLK apart
                        umma_bf16_ss(d_tmem, ad, ((uint64_t)b_hi32 << 32) | (bh_lo0 + k * 128), idesc, k == 0 ? 0u : 1u);
                        umma_bf16_ss(d_tmem, ad, ((uint64_t)b_hi32 << 32) | (bh_lo0 + ((D / 64) * (C::WBLK >> 4)) + k * 128), idesc, 1u);
                    }
                    umma_commit(&xempty[st.idx]);
                    umma_commit(&accfull[ac.idx]);
                    st.next();
                    ac.next();
                }
                umma_commit(wfree);
                ++uc;
                cur.next_unit(n_units, n_maps, n_tiles, P.n_splits);
            }
        }
    } else if (warp < 2 + C::EPI_WARPS) {
        // ================================ epilogue warps ================================
        const int q = warp & 3;                 // tensor-memory lane quarter of this warp
        const int row = q * 32 + lane;          // token row inside the tile
        constexpr int NSET = C::EPI_WARPS / 4;  // sets of four warps; a set takes the column groups c = set, set + NSET, ..
        const int set = (warp - 2) >> 2;
        ApIter cur;
        cur.start(n_units, n_maps, n_tiles, P.n_splits);
        Ring<C::NACC> ac;
        Ring<C::NO> ob;
        uint32_t uc = 0;
        const bool storer = (warp == 2 && lane == 0);
        Ring<C::NO> oldest;          // storer only: oldest output tile whose store may still be reading
        int pending = 0;
        while (cur.u < n_units) {
            const int m = cur.m;
            const int comp = m / (a.Lt * a.Ht), l = (m / a.Ht) % a.Lt, h = m % a.Ht;
            const CUtensorMap *omap = comp ? &P.out_v : &P.out_k;
            if (!mbar_wait_warp(wready, uc & 1, abort_flag, lane)) goto teardown;      // bias is in shared memory
            for (int tile = cur.tile; tile < cur.tile1; ++tile) {
                const int tok = tile * C::TT + row;
                const bool rope_unit = ROPE && comp == 0;
                // the row's position is requested before the wait for the accumulator
                int pos = 0;
                if (rope_unit && tok < a.n_tokens) pos = __ldg(P.rope.pos + tok);
                if (!mbar_wait_warp(&accfull[ac.idx], ac.phase, abort_flag, lane)) goto teardown;
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + ac.idx * C::AW;
                if (rope_unit) {
                    // forward rotation by the target model's angles: columns i and i + D/2 are a pair
                    uint8_t *ot = os + (size_t)ob.idx * C::O_BYTES;
                    float *orow = reinterpret_cast<float *>(a.out_k) + (long long)l * a.o_sl + (long long)tok * a.o_st + (long long)h * a.o_sh;
                    if (out_bf16 && !mbar_wait_warp(&ofree[ob.idx], ob.phase ^ 1, abort_flag, lane)) goto teardown;
#pragma unroll 1
                    for (int c = set; c < D / 64; c += NSET) {
                        uint32_t rl[32], rh[32];
                        {
                            tmem_ld_32x32(taddr + c * 32, rl);
                            tmem_ld_32x32(taddr + D / 2 + c * 32, rh);
                            tmem_wait_ld();
                        }
                        float ol[32], oh[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int i = c * 32 + j;
                            float cs, sn;
                            rope_cs(P.rope.f_tgt[i], pos, cs, sn);
                            const float vl = __uint_as_float(rl[j]) + bias[i], vh = __uint_as_float(rh[j]) + bias[D / 2 + i];
                            ol[j] = fmaf(vl, cs, -vh * sn);
                            oh[j] = fmaf(vl, sn, vh * cs);
                        }
                        if (out_bf16) {
#pragma unroll
                            for (int v = 0; v < 4; ++v) {
                                const int nl = c * 32 + v * 8, nh = D / 2 + nl;
                                const uint4 pl = make_uint4(pack_bf16x2(ol[v * 8 + 0], ol[v * 8 + 1]), pack_bf16x2(ol[v * 8 + 2], ol[v * 8 + 3]),
                                                            pack_bf16x2(ol[v * 8 + 4], ol[v * 8 + 5]), pack_bf16x2(ol[v * 8 + 6], ol[v * 8 + 7]));
                                const uint4 ph = make_uint4(pack_bf16x2(oh[v * 8 + 0], oh[v * 8 + 1]), pack_bf16x2(oh[v * 8 + 2], oh[v * 8 + 3]),
                                                            pack_bf16x2(oh[v * 8 + 4], oh[v * 8 + 5]), pack_bf16x2(oh[v * 8 + 6], oh[v * 8 + 7]));
                                *reinterpret_cast<uint4 *>(ot + (nl >> 6) * C::XBLK + row * 128 + ((((nl & 63) >> 3) ^ (row & 7)) << 4)) = pl;
                                *reinterpret_cast<uint4 *>(ot + (nh >> 6) * C::XBLK + row * 128 + ((((nh & 63) >> 3) ^ (row & 7)) << 4)) = ph;
                            }
                        } else if (tok < a.n_tokens) {
#pragma unroll
                            for (int v = 0; v < 8; ++v) {
                                *reinterpret_cast<float4 *>(orow + c * 32 + v * 4) = make_float4(ol[v * 4], ol[v * 4 + 1], ol[v * 4 + 2], ol[v * 4 + 3]);
                                *reinterpret_cast<float4 *>(orow + D / 2 + c * 32 + v * 4) = make_float4(oh[v * 4], oh[v * 4 + 1], oh[v * 4 + 2], oh[v * 4 + 3]);
                            }
                        }
                    }
                    tc_fence_before();
                    if (out_bf16) fence_async_smem();
                    __syncwarp();
                    if (lane == 0) { mbar_arrive(&accempty[ac.idx]); if (out_bf16) mbar_arrive(&owritten[ob.idx]); }
                    if (out_bf16) {
                        if (storer) {
                            if (mbar_wait(&owritten[ob.idx], ob.phase, abort_flag)) {
                                tma_store_5d(omap, ot, 0, tile * C::TT, 0, h, l);
                                tma_store_commit();
                                if (pending == C::NO - 1) {
                                    tma_store_wait_read_keep<C::NO - 1>();
                                    mbar_arrive(&ofree[oldest.idx]);
                                    oldest.next();
                                } else {
                                    ++pending;
                                }
                            }
                        }
                        ob.next();
                    }
                } else if (out_bf16) {
                    uint8_t *ot = os + (size_t)ob.idx * C::O_BYTES;
                    if (!mbar_wait_warp(&ofree[ob.idx], ob.phase ^ 1, abort_flag, lane)) goto teardown;
#pragma unroll 1
                    for (int c = set; c < D / 32; c += NSET) {
                        uint32_t r[32];
                        {
                            tmem_ld_32x32(taddr + c * 32, r);
                            tmem_wait_ld();
                        }
#pragma unroll
                        for (int v = 0; v < 4; ++v) {           // 4 chunks of 8 channels
                            const int n0 = c * 32 + v * 8;
                            uint4 pk;
                            pk.x = pack_bf16x2(__uint_as_float(r[v * 8 + 0]) + bias[n0 + 0], __uint_as_float(r[v * 8 + 1]) + bias[n0 + 1]);
                            pk.y = pack_bf16x2(__uint_as_float(r[v * 8 + 2]) + bias[n0 + 2], __uint_as_float(r[v * 8 + 3]) + bias[n0 + 3]);
                            pk.z = pack_bf16x2(__uint_as_float(r[v * 8 + 4]) + bias[n0 + 4], __uint_as_float(r[v * 8 + 5]) + bias[n0 + 5]);
                            pk.w = pack_bf16x2(__uint_as_float(r[v * 8 + 6]) + bias[n0 + 6], __uint_as_float(r[v * 8 + 7]) + bias[n0 + 7]);
                            const int blk = n0 >> 6, chunk = (n0 & 63) >> 3;
                            *reinterpret_cast<uint4 *>(ot + blk * C::XBLK + row * 128 + ((chunk ^ (row & 7)) << 4)) = pk;
                        }
                    }
                    tc_fence_before();
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) { mbar_arrive(&accempty[ac.idx]); mbar_arrive(&owritten[ob.idx]); }
                    if (storer) {
                        // free the tile whose store was issued NO - 1 tiles ago, then issue this tile's store
                        if (mbar_wait(&owritten[ob.idx], ob.phase, abort_flag)) {
                            tma_store_5d(omap, ot, 0, tile * C::TT, 0, h, l);
                            tma_store_commit();
                            if (pending == C::NO - 1) {
                                tma_store_wait_read_keep<C::NO - 1>();
                                mbar_arrive(&ofree[oldest.idx]);
                                oldest.next();
                            } else {
                                ++pending;
                            }
                        }
                    }
                    ob.next();
                } else {
                    float *orow = reinterpret_cast<float *>(comp ? a.out_v : a.out_k) +
                                  (long long)l * a.o_sl + (long long)tok * a.o_st + (long long)h * a.o_sh;
#pragma unroll 1
                    for (int c = set; c < D / 32; c += NSET) {
                        uint32_t r[32];
                        {
                            tmem_ld_32x32(taddr + c * 32, r);
                            tmem_wait_ld();
                        }
                        if (tok < a.n_tokens) {
#pragma unroll
                            for (int v = 0; v < 8; ++v) {
                                const int n0 = c * 32 + v * 4;
                                *reinterpret_cast<float4 *>(orow + n0) =
                                    make_float4(__uint_as_float(r[v * 4 + 0]) + bias[n0 + 0], __uint_as_float(r[v * 4 + 1]) + bias[n0 + 1],
                                                __uint_as_float(r[v * 4 + 2]) + bias[n0 + 2], __uint_as_float(r[v * 4 + 3]) + bias[n0 + 3]);
                            }
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&accempty[ac.idx]);
                }
                ac.next();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bfree);
            ++uc;
            cur.next_unit(n_units, n_maps, n_tiles, P.n_splits);
        }
        if (storer) tma_store_wait_all();          // remaining tiles need no release: nobody waits for them
    } else {
        // ================================ W conversion warps ================================
        const int ct = tid - (2 + C::EPI_WARPS) * 32;                 // 0 .. CONV_WARPS*32-1
        constexpr int CT = C::CONV_WARPS * 32;
        ApIter cur;
        cur.start(n_units, n_maps, n_tiles, P.n_splits);
        uint32_t uc = 0;
        Ring<C::NS> st;                                             // ROPE: follows the producer's ring
        // ROPE: this thread rotates the pair of 16-byte chunks (lc, lc + half a row) of RB consecutive rows.  Along
        // consecutive positions the angle of a frequency advances by a fixed step, so (cos, sin) of the next row follow
        // from the current ones by one rotation with the thread's constants (cos, sin)(theta_i); the special-function
        // unit is only needed at the first row and where the positions do not advance by one.  Packed fp32 pairs.
        constexpr int HC = D / 16, RB = C::TT / (CT / HC);
        const int lc = ct % HC, r0 = (ct / HC) * RB;
        uint32_t fsrc[8];
        uint64_t stc2[4] = {0ull, 0ull, 0ull, 0ull}, sts2[4] = {0ull, 0ull, 0ull, 0ull}, nsts2[4] = {0ull, 0ull, 0ull, 0ull};
        if (ROPE) {
            static_assert(RB <= HC, "the lanes that share a row block trade its positions");
#pragma unroll
            for (int e = 0; e < 8; ++e) fsrc[e] = P.rope.f_src[lc * 8 + e];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float c0, s0, c1, s1;
                rope_cs(fsrc[2 * e], 1, c0, s0);
                rope_cs(fsrc[2 * e + 1], 1, c1, s1);
                stc2[e] = f2_pack(c0, c1); sts2[e] = f2_pack(s0, s1); nsts2[e] = f2_pack(-s0, -s1);
            }
        }
        while (cur.u < n_units) {
            const float *Wm = a.Wb + (size_t)cur.m * (D + 1) * D;
            const bool rope_unit = ROPE && cur.m < a.Lt * a.Ht;
            // the previous unit's last MMA has read W, and its epilogues have read the bias
            if (!mbar_wait_warp(wfree, (uc & 1) ^ 1, abort_flag, lane)) goto teardown;
            if (!mbar_wait_warp(bfree, (uc & 1) ^ 1, abort_flag, lane)) goto teardown;
            for (int i = ct; i < D * (D / 8); i += CT) {              // (input channel k, chunk of 8 output channels)
                const int k = i / (D / 8), n0 = (i % (D / 8)) * 8;
                const float4 f0 = __ldg(reinterpret_cast<const float4 *>(Wm + (size_t)k * D + n0));
                const float4 f1 = __ldg(reinterpret_cast<const float4 *>(Wm + (size_t)k * D + n0 + 4));
                const float f[8] = {f0.x, f0.y, f0.z, f0.w, f1.x, f1.y, f1.z, f1.w};
                unsigned hi[4], lo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (rope_unit) {                                  // fp16 hi + lo
                        hi[e] = ap_pack_f16x2(f[2 * e], f[2 * e + 1]);
                        const float2 hf = __half22float2(*reinterpret_cast<const __half2 *>(&hi[e]));
                        lo[e] = ap_pack_f16x2(f[2 * e] - hf.x, f[2 * e + 1] - hf.y);
                        continue;
                    }
                    hi[e] = pack_bf16x2(f[2 * e], f[2 * e + 1]);
                    const float h0 = __uint_as_float(hi[e] << 16), h1 = __uint_as_float(hi[e] & 0xffff0000u);
                    lo[e] = pack_bf16x2(f[2 * e] - h0, f[2 * e + 1] - h1);
                }
                const int off = (n0 >> 6) * C::WBLK + k * 128 + ((((n0 & 63) >> 3) ^ (k & 7)) << 4);
                *reinterpret_cast<uint4 *>(whi + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<uint4 *>(wlo + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
            for (int n = ct; n < D; n += CT) bias[n] = __ldg(Wm + (size_t)D * D + n);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(wready);
            ++uc;
            if (ROPE) {
                for (int tile = cur.tile; tile < cur.tile1; ++tile) {
                    // the rows' positions are requested before the wait for the tile (their latency hides behind it):
                    // the HC lanes that share the rows r0 .. r0 + RB - 1 load one position each and trade them below
                    int mypos = 0;
                    if (rope_unit) {
                        const int tok = tile * C::TT + r0 + (lc < RB ? lc : 0);
                        mypos = (tok < a.n_tokens) ? __ldg(P.rope.pos + tok) : 0;
                    }
                    if (!mbar_wait_warp(&xfull[st.idx], st.phase, abort_flag, lane)) goto teardown;
                    if (rope_unit) {
                        uint8_t *xt = xs + st.idx * C::X_BYTES;
                        uint64_t cs2[4], sn2[4];           // packed pairs of frequencies (2 e, 2 e + 1)
                        const uint64_t neg1 = f2_pack(-1.f, -1.f);
                        int posv[RB];
#pragma unroll
                        for (int i = 0; i < RB; ++i) posv[i] = __shfl_sync(0xffffffffu, mypos, (lane & ~(HC - 1)) + i);
                        // decided once per tile, so that the row loop of the common case is straight-line code
                        bool contig = true;
#pragma unroll
                        for (int i = 1; i < RB; ++i) contig = contig && (posv[i] == posv[0] + i);
                        contig = __all_sync(0xffffffffu, contig);      // one path per warp: the general one trades lanes
                        auto first_angles = [&](int pos) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                float c0, s0, c1, s1;
                                rope_cs(fsrc[2 * e], pos, c0, s0);
                                rope_cs(fsrc[2 * e + 1], pos, c1, s1);
                                cs2[e] = f2_pack(c0, c1); sn2[e] = f2_pack(s0, s1);
                            }
                        };
                        auto next_angles = [&]() {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const uint64_t c1 = f2_fma(cs2[e], stc2[e], f2_mul(sn2[e], nsts2[e]));
                                sn2[e] = f2_fma(sn2[e], stc2[e], f2_mul(cs2[e], sts2[e]));
                                cs2[e] = c1;
                            }
                        };
                        auto rotate_row = [&](int r) {
                            const int olo = r * 128 + ((lc ^ (r & 7)) << 4);
                            const int ohi = (D == 128) ? C::XBLK + olo : r * 128 + (((lc + 4) ^ (r & 7)) << 4);
                            const uint4 vl = *reinterpret_cast<const uint4 *>(xt + olo);
                            const uint4 vh = *reinterpret_cast<const uint4 *>(xt + ohi);
                            const unsigned ul[4] = {vl.x, vl.y, vl.z, vl.w}, uh[4] = {vh.x, vh.y, vh.z, vh.w};
                            unsigned wl[4], wh[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                // rotation by -phi:  x~_i = x_i c + x_{i+D/2} s,  x~_{i+D/2} = x_{i+D/2} c - x_i s
                                const uint64_t l2 = f2_from_bf16x2(ul[e]), h2 = f2_from_bf16x2(uh[e]);
                                const uint64_t nl = f2_fma(l2, cs2[e], f2_mul(h2, sn2[e]));
                                const uint64_t nh = f2_fma(h2, cs2[e], f2_mul(f2_mul(l2, sn2[e]), neg1));
                                float a0, a1;
                                f2_unpack(nl, a0, a1); wl[e] = ap_pack_f16x2(a0, a1);
                                f2_unpack(nh, a0, a1); wh[e] = ap_pack_f16x2(a0, a1);
                            }
                            *reinterpret_cast<uint4 *>(xt + olo) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
                            *reinterpret_cast<uint4 *>(xt + ohi) = make_uint4(wh[0], wh[1], wh[2], wh[3]);
                        };
                        first_angles(posv[0]);
                        if (contig) {
#pragma unroll
                            for (int i = 0; i < RB; ++i) {
                                if (i > 0) next_angles();
                                rotate_row(r0 + i);
                            }
                        } else {
                            rotate_row(r0);
#pragma unroll 1
                            for (int i = 1; i < RB; ++i) {
                                const int pos = __shfl_sync(0xffffffffu, mypos, (lane & ~(HC - 1)) + i);
                                const int prev = __shfl_sync(0xffffffffu, mypos, (lane & ~(HC - 1)) + i - 1);
                                if (pos == prev + 1) next_angles();
                                else first_angles(pos);
                                rotate_row(r0 + i);
                            }
                        }
                        fence_async_smem();
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&xrot[st.idx]);
                    st.next();
                }
            }
            cur.next_unit(n_units, n_maps, n_tiles, P.n_splits);
        }
    }

teardown:
    __syncwarp();
    if (*abort_flag) {
        // give copies that may still be in flight time to land before the block's shared memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    // after the barrier every thread's verdict is in: a thread that finished its own role early may have passed the
    // check above before another thread gave up
    if (tid == 0 && *abort_flag && a.status) atomicExch(a.status, DEV_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

template <int D, bool ROPE>
static cudaError_t launch_ap(const ApParams &P, cudaStream_t st)
{
    using C = ApCfg<D, ROPE ? ROPE_EPI_WARPS : 4>;
    static bool attr[MAX_DEVICES] = {};
    {
        cudaError_t e = opt_in_smem(k_apply_tc<D, ROPE>, (size_t)((int)C::SMEM_BYTES), attr);
        if (e != cudaSuccess) return e;
    }
    const int n_units = 2 * P.a.Lt * P.a.Ht * P.n_splits;
    const int grid = n_units < device_sm_count() ? n_units : device_sm_count();
    k_apply_tc<D, ROPE><<<grid, C::THREADS, C::SMEM_BYTES, st>>>(P);
    return cudaGetLastError();
}

cudaError_t launch_apply_tc(const ApplyArgs &a, int d, const cb_kv_view *src, cudaStream_t st)
{
    ApParams P;
    P.a = a;
    const int TT = 128;
    const int n_maps = 2 * a.Lt * a.Ht;
    const int n_tiles = (a.n_tokens + TT - 1) / TT;
    int splits = (n_maps >= device_sm_count()) ? 1 : (device_sm_count() + n_maps - 1) / n_maps;
    if (splits > n_tiles) splits = n_tiles;
    if (splits < 1) splits = 1;
    P.n_splits = splits;
    if (!make_kv_tensor_map(&P.src_k, src->k, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                            src->stride_token, src->stride_layer, TT) ||
        !make_kv_tensor_map(&P.src_v, src->v, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                            src->stride_token, src->stride_layer, TT))
        return cudaErrorInvalidValue;
    if (a.out_dtype == CB_DTYPE_BF16) {
        if (!make_kv_tensor_map(&P.out_k, a.out_k, d, a.Ht, a.n_tokens, a.Lt, a.o_sh, a.o_st, a.o_sl, TT) ||
            !make_kv_tensor_map(&P.out_v, a.out_v, d, a.Ht, a.n_tokens, a.Lt, a.o_sh, a.o_st, a.o_sl, TT))
            return cudaErrorInvalidValue;
    } else {
        P.out_k = P.src_k;   // unused for fp32 output
        P.out_v = P.src_v;
    }
    P.rope = RopeDev{};
    cudaError_t e;
    if (a.rope_pos) {
        P.rope.pos = a.rope_pos;
        rope_frequencies(a.rope_base_src, d, P.rope.f_src);
        rope_frequencies(a.rope_base_tgt, d, P.rope.f_tgt);
        P.rope.same = (a.rope_base_src == a.rope_base_tgt) ? 1 : 0;
        e = (d == 128) ? launch_ap<128, true>(P, st) : launch_ap<64, true>(P, st);
    } else {
        e = (d == 128) ? launch_ap<128, false>(P, st) : launch_ap<64, false>(P, st);
    }
    if (e == cudaSuccess) count_launch();
    return e;
}

// =====================================================================================================================
// Apply for the head-local support over k > 1 selected layers:  out[t] = sum_f x_f[t] W_f + b, where x_f is source
// head a(h) of layer S_l[f] and W_f the f-th d x d block of the map.  W is split into bf16 hi + lo and laid out for the
// tensor core once by a preparation kernel (into the caller's workspace).  The main kernel works on groups of four
// 128-token tiles whose accumulators fill the tensor memory: per f one W block (64 KB, one bulk copy) is staged ONCE
// for the group and multiplied with the group's four source tiles (TMA), so the W traffic from L2 per tile is a
// quarter of what one tile at a time would need (that version was bound by it: 96 KB staged per 32 KB source tile).
// The loop runs f outer, tile inner; the tiles of a group finish one after the other in the last f pass and the next
// group starts with tile 0 again, so the epilogue of a group overlaps the next group's products accumulator by
// accumulator.  What bounds it: shared-memory bandwidth.  Every product reads both operands from shared memory (4 KB
// of the source tile and 4 KB of W per 128 x 128 x 16 product, i.e. 128 bytes per clock at the tensor cores' full
// rate) beside the copies that fill the stages; measured: half the tensor cores' rate.  Staging 64-channel pieces
// instead of whole tiles (deeper rings, twice the barrier traffic per product) measured 15 % slower.
// bf16 rows go from registers straight to global memory (256 contiguous bytes per thread; this path is
// bound by the tensor cores, not by its stores).
// =====================================================================================================================
template <int D>
struct MlCfg {
    static constexpr int TT = 128;
    static constexpr int NB = D / 64;
    static constexpr int XBLK = TT * 128;
    static constexpr int X_BYTES = NB * XBLK;            // one source tile
    static constexpr int WBLK = D * 128;
    static constexpr int W_BYTES = NB * WBLK;            // hi (or lo) image of one d x d block of W
    static constexpr int WSTAGE = 2 * W_BYTES;           // hi + lo
    static constexpr int GT = 4;                         // token tiles per group = accumulators in tensor memory
    static constexpr int NXS = 3, NWS = 2;               // source-tile stages, W-block stages
    static constexpr int TMEM_COLS = (GT * D < 32) ? 32 : GT * D;
    static constexpr int EPI_WARPS = 8;                  // two sets of four: tiles of a group alternate between them
    static constexpr int THREADS = (2 + EPI_WARPS) * 32;
    static constexpr size_t SMEM_BYTES = 1024 + (size_t)NXS * X_BYTES + (size_t)NWS * WSTAGE + 256;
};

struct MlParams {
    CUtensorMap src_k, src_v;
    ApplyArgs a;                 // src_layer / src_head arrays unused except src_head
    const uint8_t *wsplit;       // [n_maps][k][hi | lo][W_BYTES]
    const int *layer_sets;       // device [Lt][k]
    const int *f_order;          // device [Lt][k]: the order in which a map of target layer l walks its k blocks
    int k, n_splits;
};

// One block per (map, f): split the f-th d x d block of W into bf16 hi + lo in the swizzled MN-major layout.
template <int D>
__global__ void __launch_bounds__(256) k_w_split(const float *__restrict__ Wb, uint8_t *__restrict__ wsplit, int k)
{
    using C = MlCfg<D>;
    const int m = blockIdx.x / k, f = blockIdx.x % k;
    const float *Wm = Wb + ((size_t)m * (k * D + 1) + (size_t)f * D) * D;
    uint8_t *dst = wsplit + ((size_t)m * k + f) * 2 * C::W_BYTES;
    for (int i = threadIdx.x; i < D * (D / 8); i += 256) {
        const int kk = i / (D / 8), n0 = (i % (D / 8)) * 8;
        const float4 f0 = __ldg(reinterpret_cast<const float4 *>(Wm + (size_t)kk * D + n0));
        const float4 f1 = __ldg(reinterpret_cast<const float4 *>(Wm + (size_t)kk * D + n0 + 4));
        const float v[8] = {f0.x, f0.y, f0.z, f0.w, f1.x, f1.y, f1.z, f1.w};
        unsigned hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            hi[e] = pack_bf16x2(v[2 * e], v[2 * e + 1]);
            lo[e] = pack_bf16x2(v[2 * e] - __uint_as_float(hi[e] << 16), v[2 * e + 1] - __uint_as_float(hi[e] & 0xffff0000u));
        }
        const int off = (n0 >> 6) * C::WBLK + kk * 128 + ((((n0 & 63) >> 3) ^ (kk & 7)) << 4);
        *reinterpret_cast<uint4 *>(dst + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4 *>(dst + C::W_BYTES + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    }
}

template <int D>
__global__ void __launch_bounds__(MlCfg<D>::THREADS, 1) k_apply_ml_tc(const __grid_constant__ MlParams P)
{
    using C = MlCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *xs = smem;                                     // [NXS][X_BYTES]
    uint8_t *wsm = xs + (size_t)C::NXS * C::X_BYTES;        // [NWS][hi W_BYTES | lo W_BYTES]
    uint64_t *bars = reinterpret_cast<uint64_t *>(wsm + (size_t)C::NWS * C::WSTAGE);
    uint64_t *xfull = bars, *xempty = xfull + C::NXS;
    uint64_t *wfull = xempty + C::NXS, *wempty = wfull + C::NWS;
    uint64_t *accfull = wempty + C::NWS, *accempty = accfull + C::GT;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(accempty + C::GT);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const ApplyArgs &a = P.a;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_maps = 2 * a.Lt * a.Ht, k = P.k;
    const int n_units = n_maps * P.n_splits;
    const int n_tiles = (a.n_tokens + C::TT - 1) / C::TT;
    const bool out_bf16 = a.out_dtype == CB_DTYPE_BF16;

    if (tid == 0) {
        for (int i = 0; i < C::NXS; ++i) { mbar_init(&xfull[i], 1); mbar_init(&xempty[i], 1); }
        for (int i = 0; i < C::NWS; ++i) { mbar_init(&wfull[i], 1); mbar_init(&wempty[i], 1); }
        for (int i = 0; i < C::GT; ++i) { mbar_init(&accfull[i], 1); mbar_init(&accempty[i], 4); }
        abort_flag[0] = 0;
        abort_flag[1] = (int)P.a.poll_limit;
        mbar_fence_init();
        tma_prefetch_desc(&P.src_k); tma_prefetch_desc(&P.src_v);
    }
    if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0 && !a.starve) {   // producer: per (group, f) the W block, then the group's source tiles
            ApIter cur;
            cur.start(n_units, n_maps, n_tiles, P.n_splits);
            Ring<C::NXS> xr;
            Ring<C::NWS> wr;
            while (cur.u < n_units) {
                const int m = cur.m;
                const int comp = m / (a.Lt * a.Ht), l = (m / a.Ht) % a.Lt, h = m % a.Ht;
                const CUtensorMap *map = comp ? &P.src_v : &P.src_k;
                const int g = a.src_head[h];
                const uint8_t *wm = P.wsplit + (size_t)m * k * C::WSTAGE;
                for (int t0 = cur.tile; t0 < cur.tile1; t0 += C::GT) {
                    const int ng = min(C::GT, cur.tile1 - t0);
                    for (int f = 0; f < k; ++f) {
                        if (!mbar_wait(&wempty[wr.idx], wr.phase ^ 1, abort_flag)) goto ml_teardown;
                        mbar_arrive_expect_tx(&wfull[wr.idx], C::WSTAGE);
                        const int fb = P.f_order[l * k + f];          // block of this step (see launch_apply_ml_tc)
                        bulk_load(wsm + (size_t)wr.idx * C::WSTAGE, wm + (size_t)fb * C::WSTAGE, C::WSTAGE, &wfull[wr.idx]);
                        wr.next();
                        const int j = P.layer_sets[l * k + fb];
                        for (int t = 0; t < ng; ++t) {
                            if (!mbar_wait(&xempty[xr.idx], xr.phase ^ 1, abort_flag)) goto ml_teardown;
                            mbar_arrive_expect_tx(&xfull[xr.idx], C::X_BYTES);
                            tma_load_5d(xs + (size_t)xr.idx * C::X_BYTES, map, &xfull[xr.idx], 0, (t0 + t) * C::TT, 0, g, j);
                            xr.next();
                        }
                    }
                }
                cur.next_unit(n_units, n_maps, n_tiles, P.n_splits);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {          // MMA issuer
            constexpr uint32_t idesc = umma_idesc_bf16(128, D, false, true);
            const uint64_t proto_a = umma_smem_desc_sw128(0, 16, 1024);
            const uint64_t proto_b = umma_smem_desc_sw128(0, C::WBLK, 1024);
            const uint32_t a_hi32 = (uint32_t)(proto_a >> 32), b_hi32 = (uint32_t)(proto_b >> 32);
            const uint32_t a_lo0 = (uint32_t)proto_a | ((smem_u32(xs) & 0x3FFFFu) >> 4);
            const uint32_t b_lo0 = (uint32_t)proto_b | ((smem_u32(wsm) & 0x3FFFFu) >> 4);
            ApIter cur;
            cur.start(n_units, n_maps, n_tiles, P.n_splits);
            Ring<C::NXS> xr;
            Ring<C::NWS> wr;
            uint32_t accphase = 0;          // bit t: phase of accumulator t
            while (cur.u < n_units) {
                for (int t0 = cur.tile; t0 < cur.tile1; t0 += C::GT) {
                    const int ng = min(C::GT, cur.tile1 - t0);
                    for (int f = 0; f < k; ++f) {
                        if (!mbar_wait(&wfull[wr.idx], wr.phase, abort_flag)) goto ml_teardown;
                        const uint32_t bl = b_lo0 + wr.idx * (C::WSTAGE >> 4);
                        for (int t = 0; t < ng; ++t) {
                            if (f == 0 && !mbar_wait(&accempty[t], ((accphase >> t) & 1) ^ 1, abort_flag)) goto ml_teardown;
                            if (!mbar_wait(&xfull[xr.idx], xr.phase, abort_flag)) goto ml_teardown;
                            tc_fence_after();
                            const uint32_t d_tmem = tmem_base + t * D;
                            const uint32_t al = a_lo0 + xr.idx * (C::X_BYTES >> 4);
#pragma unroll
                            for (int kk = 0; kk < D / 16; ++kk) {
                                const uint64_t ad = ((uint64_t)a_hi32 << 32) | (al + (kk >> 2) * (C::XBLK >> 4) + (kk & 3) * 2);
                                umma_bf16_ss(d_tmem, ad, ((uint64_t)b_hi32 << 32) | (bl + kk * 128), idesc, (f == 0 && kk == 0) ? 0u : 1u);
                                umma_bf16_ss(d_tmem, ad, ((uint64_t)b_hi32 << 32) | (bl + (C::W_BYTES >> 4) + kk * 128), idesc, 1u);
                            }
                            umma_commit(&xempty[xr.idx]);
                            xr.next();
                            if (f == k - 1) { umma_commit(&accfull[t]); accphase ^= 1u << t; }
                        }
                        umma_commit(&wempty[wr.idx]);
                        wr.next();
                    }
                }
                cur.next_unit(n_units, n_maps, n_tiles, P.n_splits);
            }
        }
    } else {
        // epilogue warps: tensor memory -> + bias -> bf16 or fp32 rows straight to global memory; warps 2..5 take the
        // even tiles of a group, warps 6..9 the odd ones
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const int eset = (warp - 2) >> 2;
        ApIter cur;
        cur.start(n_units, n_maps, n_tiles, P.n_splits);
        uint32_t accphase = 0;
        while (cur.u < n_units) {
            const int m = cur.m;
            const int comp = m / (a.Lt * a.Ht), l = (m / a.Ht) % a.Lt, h = m % a.Ht;
            const float *bias = a.Wb + ((size_t)m * (k * D + 1) + (size_t)k * D) * D;     // last row of the map
            for (int t0 = cur.tile; t0 < cur.tile1; t0 += C::GT) {
                const int ng = min(C::GT, cur.tile1 - t0);
                for (int t = eset; t < ng; t += 2) {
                    if (!mbar_wait_warp(&accfull[t], (accphase >> t) & 1, abort_flag, lane)) goto ml_teardown;
                    accphase ^= 1u << t;
                    tc_fence_after();
                    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + t * D;
                    const int tok = (t0 + t) * C::TT + row;
                    const long long off = (long long)l * a.o_sl + (long long)tok * a.o_st + (long long)h * a.o_sh;
#pragma unroll 1
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t r[32];
                        tmem_ld_32x32(taddr + c * 32, r);
                        tmem_wait_ld();
                        if (c == D / 32 - 1) {          // the accumulator is in registers: the next group may reuse it
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&accempty[t]);
                        }
                        if (tok >= a.n_tokens) continue;
                        if (out_bf16) {
                            __nv_bfloat16 *orow = reinterpret_cast<__nv_bfloat16 *>(comp ? a.out_v : a.out_k) + off;
#pragma unroll
                            for (int v = 0; v < 4; ++v) {
                                const int n0 = c * 32 + v * 8;
                                const float4 b0 = __ldg(reinterpret_cast<const float4 *>(bias + n0));
                                const float4 b1 = __ldg(reinterpret_cast<const float4 *>(bias + n0 + 4));
                                uint4 pk;
                                pk.x = pack_bf16x2(__uint_as_float(r[v * 8 + 0]) + b0.x, __uint_as_float(r[v * 8 + 1]) + b0.y);
                                pk.y = pack_bf16x2(__uint_as_float(r[v * 8 + 2]) + b0.z, __uint_as_float(r[v * 8 + 3]) + b0.w);
                                pk.z = pack_bf16x2(__uint_as_float(r[v * 8 + 4]) + b1.x, __uint_as_float(r[v * 8 + 5]) + b1.y);
                                pk.w = pack_bf16x2(__uint_as_float(r[v * 8 + 6]) + b1.z, __uint_as_float(r[v * 8 + 7]) + b1.w);
                                *reinterpret_cast<uint4 *>(orow + n0) = pk;
                            }
                        } else {
                            float *orow = reinterpret_cast<float *>(comp ? a.out_v : a.out_k) + off;
#pragma unroll
                            for (int v = 0; v < 8; ++v) {
                                const int n0 = c * 32 + v * 4;
                                const float4 b0 = __ldg(reinterpret_cast<const float4 *>(bias + n0));
                                *reinterpret_cast<float4 *>(orow + n0) =
                                    make_float4(__uint_as_float(r[v * 4 + 0]) + b0.x, __uint_as_float(r[v * 4 + 1]) + b0.y,
                                                __uint_as_float(r[v * 4 + 2]) + b0.z, __uint_as_float(r[v * 4 + 3]) + b0.w);
                            }
                        }
                    }
                }
                // accumulators this set does not drain still change phase for the next group
                for (int t = 1 - eset; t < ng; t += 2) accphase ^= 1u << t;
            }
            cur.next_unit(n_units, n_maps, n_tiles, P.n_splits);
        }
    }

ml_teardown:
    __syncwarp();
    if (*abort_flag) {
        // give copies that may still be in flight time to land before the block's shared memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (tid == 0 && *abort_flag && a.status) atomicExch(a.status, DEV_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

size_t apply_ml_workspace_bytes(int n_maps, int k, int d, int Lt)
{
    return (size_t)n_maps * k * 2 * (size_t)d * d * 2 + ((sizeof(int) * 2 * (size_t)Lt * k + 255) / 256) * 256;
}

template <int D>
static cudaError_t launch_ml(const MlParams &P, const float *Wb, uint8_t *wsplit, cudaStream_t st)
{
    using C = MlCfg<D>;
    static bool attr[MAX_DEVICES] = {};
    {
        cudaError_t e = opt_in_smem(k_apply_ml_tc<D>, (size_t)((int)C::SMEM_BYTES), attr);
        if (e != cudaSuccess) return e;
    }
    const int n_maps = 2 * P.a.Lt * P.a.Ht;
    k_w_split<D><<<n_maps * P.k, 256, 0, st>>>(Wb, wsplit, P.k);
    const int n_units = n_maps * P.n_splits;
    const int grid = n_units < device_sm_count() ? n_units : device_sm_count();
    k_apply_ml_tc<D><<<grid, C::THREADS, C::SMEM_BYTES, st>>>(P);
    return cudaGetLastError();
}

cudaError_t launch_apply_ml_tc(const ApplyArgs &a, int d, int k, const int *layer_sets_host, const cb_kv_view *src,
                               void *workspace, cudaStream_t st)
{
    MlParams P;
    P.a = a;
    P.k = k;
    const int TT = 128;
    const int n_maps = 2 * a.Lt * a.Ht;
    const int n_tiles = (a.n_tokens + TT - 1) / TT;
    int splits = (n_maps >= device_sm_count()) ? 1 : (device_sm_count() + n_maps - 1) / n_maps;
    if (splits > n_tiles) splits = n_tiles;
    if (splits < 1) splits = 1;
    P.n_splits = splits;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    const size_t wbytes = (size_t)n_maps * k * 2 * (size_t)d * d * 2;
    P.wsplit = ws;
    P.layer_sets = reinterpret_cast<const int *>(ws + wbytes);
    P.f_order = P.layer_sets + (size_t)a.Lt * k;
    // Order of the k blocks of a map: by (source layer mod k).  The persistent blocks walk their units in step, and
    // maps of neighbouring target layers select overlapping source layers; with this order every map that reads
    // layer j reads it in the same step, so that one fetch from device memory serves all of them through L2 (for k
    // consecutive layers the order is a rotation of the set).  The sum over blocks does not depend on the order
    // beyond fp32 rounding, and the order is fixed by the problem.
    std::vector<int> tab(layer_sets_host, layer_sets_host + (size_t)a.Lt * k);
    tab.resize(2 * (size_t)a.Lt * k);
    for (int l = 0; l < a.Lt; ++l) {
        int *ord = tab.data() + (size_t)a.Lt * k + (size_t)l * k;
        for (int f = 0; f < k; ++f) ord[f] = f;
        const int *set = layer_sets_host + (size_t)l * k;
        std::stable_sort(ord, ord + k, [&](int x, int y) { return set[x] % k < set[y] % k; });
    }
    cudaError_t e = cudaMemcpyAsync(ws + wbytes, tab.data(), sizeof(int) * tab.size(), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return e;
    if (!make_kv_tensor_map(&P.src_k, src->k, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                            src->stride_token, src->stride_layer, TT) ||
        !make_kv_tensor_map(&P.src_v, src->v, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                            src->stride_token, src->stride_layer, TT))
        return cudaErrorInvalidValue;
    e = (d == 128) ? launch_ml<128>(P, a.Wb, ws, st) : launch_ml<64>(P, a.Wb, ws, st);
    if (e == cudaSuccess) count_launch(2);
    return e;
}

}  // namespace cb
