// Head-local weighted statistics (d = 128) with the weighted operand in TENSOR MEMORY.
//
// Same contraction as the shared-memory kernel (D[d][2d] = (w .* X)^T [X | Y] over tokens plus the bias sums), same
// units, slots and summation order of the splits.  What differs is where the first MMA operand lives: the fold warps
// write A = bf16(w x) straight into tensor memory (lane = channel, two tokens per 32-bit column) and the MMA reads it
// from there.  Per 64-token tile that saves the 16 KB shared-memory write of the weighted tile and its 16 KB read by
// the tensor cores (96 KB of shared-memory traffic instead of 128 KB) and the shared-memory space of the operand
// buffers.  On full launches the board runs into its power limit (the SM clock measured inside the kernel falls to
// about 1.43 GHz, while each part of the kernel alone runs at 1.8 - 1.96 GHz): what counts is the energy per tile.
//
//   warp 0       X tile producer (TMA); last warp: Y tile + token weights producer
//   warps 2..9   fold: a warp owns the channel quarter (warp % 4) that its tensor-memory lanes cover and one half of
//                the tile's tokens.  ldmatrix (8x8, transposed) delivers for thread i the pair (token 2j, 2j+1) of
//                channel i/4, which is exactly the register layout of the 16-lane x 128-bit tensor-memory store; the
//                swizzled tile is read without bank conflicts.
//   warp 1       MMA issuer: A from tensor memory, B = [X | Y] from shared memory (N = 256, MN-major)
//   warps 10..13 drain: tensor memory -> registers -> vector reductions onto the unit's slot (one writer per slot
//                and launch: the result does not depend on timing)
//   warps 14..   bias sums s_y = sum w y, s_w = sum w on the ALUs, in warps of their own: the MMA of a tile waits for
//                the weighted operand only.  Measured: 4 such warps 1 % faster than 8; 16 fold warps (16 channels
//                each) 4 % slower than 8.
// Tensor memory: columns 0..255 the accumulator, from 256 the ring of weighted operands (32 columns each; hi and lo
// images when compensated).  One accumulator: the MMA waits while a unit's result is read out (about 1 % of a unit).
// Every wait is bounded: if one runs out the block sets the context's status word and tears down.
#include <cudaTypedefs.h>

#ifndef CB_TS_TT
#define CB_TS_TT 128
#endif
#ifndef CB_TS_NS
#define CB_TS_NS (CB_TS_TT == 128 ? 3 : 5)
#endif
#ifndef CB_TS_NA
#define CB_TS_NA (CB_TS_TT == 128 ? 3 : 4)
#endif
#ifndef CB_TS_GSPLIT
#define CB_TS_GSPLIT 1
#endif
#ifndef CB_TS_YW
#define CB_TS_YW 8
#endif

#include "cb_internal.cuh"
#include "cb_ptx.cuh"

namespace cb {

using namespace ptx;

bool make_kv_tensor_map(CUtensorMap *map, const void *base, int d, int H, long long T, int L,
                        long long sh, long long st, long long sl, int box_tokens);

namespace {

template <bool COMP>
struct TsCfg {
    static constexpr int D = 128;
    static constexpr int TT = CB_TS_TT;               // tokens per tile
    static constexpr int BLK = TT * 128;              // one 64-channel block of a tile: TT rows of 128 bytes
    static constexpr int STAGE_BYTES = 4 * BLK;       // [X blocks 0, 1 | Y blocks 0, 1]
    static constexpr int NS = CB_TS_NS;
    static constexpr int A_PARTS = COMP ? 2 : 1;
    static constexpr int A_PART_COLS = TT / 2;        // columns of one image of the weighted operand (two tokens per column)
    static constexpr int A_COLS = A_PART_COLS * A_PARTS;
    static constexpr int NA = (CB_TS_NA * A_COLS > 256) ? 256 / A_COLS : CB_TS_NA;
    static constexpr int N = 2 * D;                   // accumulator columns
    static constexpr int A_COL0 = N;
    static constexpr int TMEM_COLS = 512;
    static constexpr int GSPLIT = CB_TS_GSPLIT;       // 2: a fold warp takes 16 of its quarter's 32 channels
    static constexpr int FOLD_WARPS = 8 * GSPLIT, DRAIN_WARPS = 4, YSUM_WARPS = CB_TS_YW;
    static constexpr int YSUM_WARP0 = 2 + FOLD_WARPS + DRAIN_WARPS;
    static constexpr int YPROD_WARP = YSUM_WARP0 + YSUM_WARPS;
    static constexpr int YSUM_THREADS = YSUM_WARPS * 32;
    static constexpr int THREADS = (YPROD_WARP + 1) * 32;
    static constexpr int RED_STRIDE = D + 4;          // per bias warp: s_y[D], s_w, pad
    static constexpr int RED_FLOATS = YSUM_WARPS * RED_STRIDE + 2 * D;   // ... then s_x of the two token halves
    static constexpr size_t SMEM_BYTES = 1024 + (size_t)NS * STAGE_BYTES + RED_FLOATS * 4 + NS * TT * 4 + 256;
    static_assert(N + NA * A_COLS <= TMEM_COLS, "tensor memory columns");
    static_assert(NA <= NS, "an operand buffer is released through its tile's stage barrier");
};

struct TsParams {
    CUtensorMap src_k, src_v, tgt_k, tgt_v;   // 5-D tiled maps: (64 channels, token, channel block, head, layer)
    AccumArgs a;
    int drain_tiles;                          // tiles accumulated in tensor memory between drains
};

// Walks the tiles of this block's units in order: units u = blockIdx.x, += gridDim.x; unit -> (map, split) -> tiles
// [tile, tile1).  Empty units are skipped.
struct UnitIter {
    int u, tile, tile1, m, split, comp, l, h, src_l, src_h;
    __device__ __forceinline__ void start(const AccumArgs &a, int n_units, int n_maps, int n_tiles)
    {
        u = (int)blockIdx.x - (int)gridDim.x;
        tile = tile1 = 0;
        next_unit(a, n_units, n_maps, n_tiles);
    }
    __device__ __forceinline__ bool valid(int n_units) const { return u < n_units; }
    __device__ __forceinline__ void next_unit(const AccumArgs &a, int n_units, int n_maps, int n_tiles)
    {
        do {
            u += gridDim.x;
            if (u >= n_units) return;
            m = u % n_maps;
            split = u / n_maps;
            tile = (int)(((long long)n_tiles * split) / a.n_splits);
            tile1 = (int)(((long long)n_tiles * (split + 1)) / a.n_splits);
        } while (tile >= tile1);
        comp = m / (a.Lt * a.Ht);
        l = (m / a.Ht) % a.Lt;
        h = m % a.Ht;
        src_l = a.src_layer[l];
        src_h = a.src_head[h];
    }
    __device__ __forceinline__ void advance(const AccumArgs &a, int n_units, int n_maps, int n_tiles)
    {
        if (++tile >= tile1) next_unit(a, n_units, n_maps, n_tiles);
    }
};

template <int N>
struct Ring {
    uint32_t idx = 0, phase = 0;
    __device__ __forceinline__ void next() { if (++idx == N) { idx = 0; phase ^= 1; } }
};

// Packed fp32 pairs (two fp32 lanes per instruction).
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t f2_from_bf16x2(unsigned u) { return f2_pack(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u)); }
__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi)
{
    unsigned r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// CEN: two-pass centred construction: the weighted operand is w (x - mu_x) with the means of P.a.mu; the slot's s_x
// entries become the column sums of the ROUNDED weighted operand (what the reduction needs for its exact correction).
template <bool COMP, bool CEN>
__global__ void __launch_bounds__(TsCfg<COMP>::THREADS, 1) k_accum_ts(const __grid_constant__ TsParams P)
{
    using C = TsCfg<COMP>;
    constexpr int D = C::D;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *xy = smem;                                       // [NS][STAGE_BYTES]
    float *red = reinterpret_cast<float *>(xy + (size_t)C::NS * C::STAGE_BYTES);
    float *redx = red + C::YSUM_WARPS * C::RED_STRIDE;        // [2 token halves][D]
    float *wst = red + C::RED_FLOATS;                         // [NS][TT] token weights of the staged tile
    uint64_t *bars = reinterpret_cast<uint64_t *>(wst + C::NS * C::TT);
    uint64_t *full = bars;                 // [NS] tile landed: X bytes (1 arrival), Y bytes (1), weights (32 lanes)
    uint64_t *empty = full + C::NS;        // [NS] stage free: MMA done (1) + every fold and bias warp done
    uint64_t *afull = empty + C::NS;       // [NA] weighted operand written to tensor memory (every fold warp)
    uint64_t *accfull = afull + C::NA;     // [1]  accumulator complete (MMA)
    uint64_t *accempty = accfull + 1;      // [1]  accumulator read out (4 drain warps)
    uint64_t *redfull = accempty + 1;      // [1]  bias partials of all fold and bias warps written
    uint64_t *reddone = redfull + 1;       // [1]  bias partials consumed
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(reddone + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const AccumArgs &a = P.a;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_maps = 2 * a.Lt * a.Ht;
    const int n_units = n_maps * a.n_splits;
    const int n_tiles = (a.n_tokens + C::TT - 1) / C::TT;

    if (tid == 0) {
        for (int i = 0; i < C::NS; ++i) { mbar_init(&full[i], 2 + 32); mbar_init(&empty[i], 1 + C::FOLD_WARPS + C::YSUM_WARPS); }
        for (int i = 0; i < C::NA; ++i) mbar_init(&afull[i], C::FOLD_WARPS);
        mbar_init(accfull, 1);
        mbar_init(accempty, C::DRAIN_WARPS);
        mbar_init(redfull, C::FOLD_WARPS + C::YSUM_WARPS);
        mbar_init(reddone, C::YSUM_WARPS);
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&P.src_k); tma_prefetch_desc(&P.src_v);
        tma_prefetch_desc(&P.tgt_k); tma_prefetch_desc(&P.tgt_v);
    }
    if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ================================ X producer (one thread) ================================
        if (lane == 0) {
            UnitIter cur;
            cur.start(a, n_units, n_maps, n_tiles);
            Ring<C::NS> st;
            while (cur.valid(n_units)) {
                const CUtensorMap *map = cur.comp ? &P.src_v : &P.src_k;
                const int g = cur.src_h, j = cur.src_l, u = cur.u;
                do {
                    if (!mbar_wait(&empty[st.idx], st.phase ^ 1, abort_flag)) goto teardown;
                    mbar_arrive_expect_tx(&full[st.idx], 2 * C::BLK);
                    tma_load_5d(xy + st.idx * C::STAGE_BYTES, map, &full[st.idx], 0, cur.tile * C::TT, 0, g, j);
                    st.next();
                    cur.advance(a, n_units, n_maps, n_tiles);
                } while (cur.u == u);
            }
        }
    } else if (warp == C::YPROD_WARP) {
        // ================================ Y + weights producer ================================
        UnitIter cur;
        cur.start(a, n_units, n_maps, n_tiles);
        Ring<C::NS> st;
        while (cur.valid(n_units)) {
            const CUtensorMap *map = cur.comp ? &P.tgt_v : &P.tgt_k;
            const int h = cur.h, l = cur.l, u = cur.u;
            const float *w = (cur.comp ? a.w_v : a.w_k) + (long long)l * a.w_sl + (long long)h * a.w_sh;
            do {
                if (!mbar_wait_warp(&empty[st.idx], st.phase ^ 1, abort_flag, lane)) goto teardown;
                const int tok0 = cur.tile * C::TT;
                if (lane == 0) {
                    mbar_arrive_expect_tx(&full[st.idx], 2 * C::BLK);
                    tma_load_5d(xy + st.idx * C::STAGE_BYTES + 2 * C::BLK, map, &full[st.idx], 0, tok0, 0, h, l);
                }
#pragma unroll
                for (int q = 0; q < C::TT / 32; ++q) {
                    const int r = lane + 32 * q;
                    const bool in = tok0 + r < a.n_tokens;
                    cp_async_4(&wst[st.idx * C::TT + r], w + (in ? tok0 + r : 0), in ? 4u : 0u);
                }
                cp_async_arrive_noinc(&full[st.idx]);
                st.next();
                cur.advance(a, n_units, n_maps, n_tiles);
            } while (cur.u == u);
        }
    } else if (warp == 1) {
        // ================================ MMA issuer (one thread) ================================
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, C::N, false, true);
            const uint64_t proto = umma_smem_desc_sw128(0, C::BLK, 1024);
            const uint32_t desc_hi = (uint32_t)(proto >> 32);
            const uint32_t b_lo0 = (uint32_t)proto | ((smem_u32(xy) & 0x3FFFFu) >> 4);
            Ring<C::NS> st;
            Ring<C::NA> ar;
            uint32_t sr = 0;
            UnitIter cur;
            cur.start(a, n_units, n_maps, n_tiles);
            while (cur.valid(n_units)) {
                const int tile1 = cur.tile1;
                for (int sr0 = cur.tile; sr0 < tile1; sr0 += P.drain_tiles, ++sr) {
                    const int n_sub = min(tile1 - sr0, P.drain_tiles);
                    if (!mbar_wait(accempty, (sr & 1) ^ 1, abort_flag)) goto teardown;
                    tc_fence_after();
                    uint32_t accum = 0;
                    for (int t = 0; t < n_sub; ++t) {
                        // afull implies full: every fold warp saw the tile land before it wrote the weighted operand
                        if (!mbar_wait(&afull[ar.idx], ar.phase, abort_flag)) goto teardown;
                        tc_fence_after();
                        const uint32_t bl = b_lo0 + st.idx * (C::STAGE_BYTES >> 4);
                        const uint32_t at = tmem_base + C::A_COL0 + ar.idx * C::A_COLS;
#pragma unroll
                        for (int k = 0; k < C::TT / 16; ++k) {
                            const uint64_t bd = ((uint64_t)desc_hi << 32) | (bl + k * 128);
                            umma_bf16_ts(tmem_base, at + k * 8, bd, idesc, k == 0 ? accum : 1u);
                            if (COMP) umma_bf16_ts(tmem_base, at + C::A_PART_COLS + k * 8, bd, idesc, 1u);
                        }
                        accum = 1;
                        umma_commit(&empty[st.idx]);     // frees the stage and (through it) the weighted-operand buffer
                        st.next();
                        ar.next();
                    }
                    umma_commit(accfull);
                }
                cur.next_unit(a, n_units, n_maps, n_tiles);
            }
        }
    } else if (warp < 2 + C::FOLD_WARPS) {
        // ================================ fold warps ================================
        const int fw = warp - 2;
        const int q = warp & 3;             // tensor-memory lane quarter = channels 32 q .. 32 q + 31
        const int hf = (fw >> 2) & 1;       // token half of the tile
        constexpr int GN = 2 / C::GSPLIT;   // 16-channel groups per warp
        const int g0 = (C::GSPLIT == 2) ? (fw >> 3) : 0;
        // ldmatrix row address of this lane: matrix j = lane / 8 is (8-channel chunk j & 1, token group j / 2), row
        // lane % 8 is a token; the 128-byte swizzle XORs the chunk index with the token's low three bits.
        const int lm_row = hf * (C::TT / 2) + 8 * (lane >> 4) + (lane & 7);
        uint32_t lm_off[GN];
#pragma unroll
        for (int g = 0; g < GN; ++g)
            lm_off[g] = (q >> 1) * C::BLK + lm_row * 128 + (((4 * (q & 1) + 2 * (g0 + g) + ((lane >> 3) & 1)) ^ (lane & 7)) << 4);
        const uint32_t a_lane = tmem_base + ((uint32_t)(q * 32) << 16) + C::A_COL0 + hf * (C::TT / 4);
        Ring<C::NS> st, old;       // `old` trails `st` by NA tiles
        Ring<C::NA> ar;
        uint32_t it = 0, uc = 0;
        UnitIter cur;
        cur.start(a, n_units, n_maps, n_tiles);
        while (cur.valid(n_units)) {
            const int m = cur.m, n_t = cur.tile1 - cur.tile;
            uint64_t sx2[GN][2];           // [16-channel group][chunk]: sums over this thread's token pairs
            uint64_t nmu2[GN][2];
#pragma unroll
            for (int g = 0; g < GN; ++g)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    sx2[g][c] = 0ull;
                    nmu2[g][c] = 0ull;
                    if (CEN) {
                        const float mu = __ldg(a.mu + (size_t)m * (2 * D + 1) + q * 32 + 16 * (g0 + g) + 8 * c + (lane >> 2));
                        nmu2[g][c] = f2_pack(-mu, -mu);
                    }
                }
            for (int t = 0; t < n_t; ++t) {
                if (!mbar_wait_warp(&full[st.idx], st.phase, abort_flag, lane)) goto teardown;
                // the operand buffer was last read by the MMAs of tile it - NA, which also release that tile's stage
                if (it >= (uint32_t)C::NA) {
                    if (!mbar_wait_warp(&empty[old.idx], old.phase, abort_flag, lane)) goto teardown;
                    old.next();
                    tc_fence_after();
                }
                const uint32_t stage_u32 = smem_u32(xy + st.idx * C::STAGE_BYTES);
                const float *wt = wst + st.idx * C::TT;
                // 32 tokens of this warp's half at a time; token pairs of this lane: + 8 j + 2 (lane % 4) + {0, 1}
#pragma unroll
                for (int sub = 0; sub < C::TT / 64; ++sub) {
                uint64_t w2[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    w2[j] = *reinterpret_cast<const uint64_t *>(wt + hf * (C::TT / 2) + sub * 32 + 8 * j + 2 * (lane & 3));
                uint32_t r[GN][2][4];
#pragma unroll
                for (int g = 0; g < GN; ++g)
#pragma unroll
                    for (int tp = 0; tp < 2; ++tp) ldmatrix_x4_trans(stage_u32 + lm_off[g] + (sub * 32 + tp * 16) * 128, r[g][tp]);
#pragma unroll
                for (int g = 0; g < GN; ++g) {
                    uint32_t oh[8], ol[8];
#pragma unroll
                    for (int tp = 0; tp < 2; ++tp) {
#pragma unroll
                        for (int mi = 0; mi < 4; ++mi) {
                            const int c = mi & 1;
                            uint64_t xf = f2_from_bf16x2(r[g][tp][mi]);
                            if (CEN) xf = f2_add(xf, nmu2[g][c]);                       // x - mu_x
                            const uint64_t pr = f2_mul(w2[2 * tp + (mi >> 1)], xf);      // w x for two tokens
                            if (!CEN) sx2[g][c] = f2_add(sx2[g][c], pr);
                            float p0, p1;
                            f2_unpack(pr, p0, p1);
                            const unsigned hw = pack_bf16x2(p0, p1);
                            oh[4 * tp + mi] = hw;
                            if (COMP) ol[4 * tp + mi] = pack_bf16x2(p0 - __uint_as_float(hw << 16), p1 - __uint_as_float(hw & 0xffff0000u));
                            if (CEN) {                                                  // sum of what the tensor cores will see
                                sx2[g][c] = f2_add(sx2[g][c], f2_from_bf16x2(hw));
                                if (COMP) sx2[g][c] = f2_add(sx2[g][c], f2_from_bf16x2(ol[4 * tp + mi]));
                            }
                        }
                    }
                    const uint32_t ta = a_lane + ((uint32_t)(16 * (g0 + g)) << 16) + ar.idx * C::A_COLS + sub * 16;
                    tmem_st_16x128_x4(ta, oh);
                    if (COMP) tmem_st_16x128_x4(ta + C::A_PART_COLS, ol);
                }
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&afull[ar.idx]); mbar_arrive(&empty[st.idx]); }
                st.next();
                ar.next();
                ++it;
            }
            // ---- s_x of this unit: the four lanes that hold a channel add up; the bias warps write the slot ----
            if (!mbar_wait_warp(reddone, (uc & 1) ^ 1, abort_flag, lane, true)) goto teardown;
#pragma unroll
            for (int g = 0; g < GN; ++g)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    float lo, hi;
                    f2_unpack(sx2[g][c], lo, hi);
                    float v = lo + hi;
                    v += __shfl_xor_sync(0xffffffffu, v, 1);
                    v += __shfl_xor_sync(0xffffffffu, v, 2);
                    if ((lane & 3) == 0) redx[hf * D + q * 32 + 16 * (g0 + g) + 8 * c + (lane >> 2)] = v;
                }
            __syncwarp();
            if (lane == 0) mbar_arrive(redfull);
            ++uc;
            cur.next_unit(a, n_units, n_maps, n_tiles);
        }
    } else if (warp >= C::YSUM_WARP0 && warp < C::YPROD_WARP) {
        // ================================ bias warps: s_y = sum w y, s_w = sum w ================================
        // thread = (16-byte chunk cc of the target row, row group rg), rows rg + 16 i.  Off the MMA's critical path.
        const int yt = tid - C::YSUM_WARP0 * 32, yw = warp - C::YSUM_WARP0;
        const int cc = yt & 15, rg = yt >> 4;
        constexpr int YRG = C::YSUM_THREADS / 16, YR = C::TT / YRG;   // row groups, rows per thread
        static_assert(YRG % 8 == 0 && YR % 4 == 0, "row groups must preserve the swizzle phase; rows go in batches of four");
        const int y_off = 2 * C::BLK + (cc >> 3) * C::BLK + rg * 128 + (((cc & 7) ^ (rg & 7)) << 4);
        Ring<C::NS> st;
        uint32_t uc = 0;
        UnitIter cur;
        cur.start(a, n_units, n_maps, n_tiles);
        while (cur.valid(n_units)) {
            const int m = cur.m, split = cur.split, n_t = cur.tile1 - cur.tile;
            uint64_t sy2[4];
            float sw = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) sy2[e] = 0ull;
            for (int t = 0; t < n_t; ++t) {
                if (!mbar_wait_warp(&full[st.idx], st.phase, abort_flag, lane)) goto teardown;
                const uint8_t *stage = xy + st.idx * C::STAGE_BYTES;
                const float *wt = wst + st.idx * C::TT;
#pragma unroll
                for (int i0 = 0; i0 < YR; i0 += 4) {
                    float wr[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) wr[i] = wt[rg + YRG * (i0 + i)];
                    if (!CEN) {
                        uint4 yv[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) yv[i] = *reinterpret_cast<const uint4 *>(stage + y_off + (i0 + i) * (YRG * 128));
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint64_t wr2 = f2_pack(wr[i], wr[i]);
                            const unsigned yu[4] = {yv[i].x, yv[i].y, yv[i].z, yv[i].w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) sy2[e] = f2_fma(wr2, f2_from_bf16x2(yu[e]), sy2[e]);
                        }
                    }
                    if (cc == 0) sw += (wr[0] + wr[1]) + (wr[2] + wr[3]);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[st.idx]);
                st.next();
            }
            if (!mbar_wait_warp(reddone, (uc & 1) ^ 1, abort_flag, lane)) goto teardown;
            {
                float sy[8];
#pragma unroll
                for (int e = 0; e < 4; ++e) f2_unpack(sy2[e], sy[2 * e], sy[2 * e + 1]);
#pragma unroll
                for (int e = 0; e < 8; ++e) sy[e] += __shfl_xor_sync(0xffffffffu, sy[e], 16);
                sw += __shfl_xor_sync(0xffffffffu, sw, 16);
                float *rw = red + yw * C::RED_STRIDE;
                if (lane < 16) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) rw[cc * 8 + e] = sy[e];
                    if (cc == 0) rw[D] = sw;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(redfull);
            if (!mbar_wait_warp(redfull, uc & 1, abort_flag, lane)) goto teardown;
            {
                float *slot = a.slots + ((size_t)split * n_maps + m) * slot_floats(D);
                for (int v = yt; v < 2 * D + 1; v += C::YSUM_THREADS) {
                    float sum = 0.f;
                    if (v < D) sum = redx[v] + redx[D + v];
                    else {
#pragma unroll
                        for (int k = 0; k < C::YSUM_WARPS; ++k) sum += red[k * C::RED_STRIDE + (v - D)];
                    }
                    slot[slot_sx(D) + v] += sum;    // s_x, s_y, s_w are adjacent in the slot
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(reddone);
            ++uc;
            cur.next_unit(a, n_units, n_maps, n_tiles);
        }
    } else {
        // ================================ drain warps ================================
        const int q = warp & 3;             // tensor-memory lane quarter this warp may access
        const int row = q * 32 + lane;      // row of D = channel of the weighted operand
        uint32_t sr = 0;
        UnitIter cur;
        cur.start(a, n_units, n_maps, n_tiles);
        while (cur.valid(n_units)) {
            float *grow = a.slots + ((size_t)cur.split * n_maps + cur.m) * slot_floats(D) + (size_t)row * C::N;
            for (int sr0 = cur.tile; sr0 < cur.tile1; sr0 += P.drain_tiles, ++sr) {
                if (!mbar_wait_warp(accfull, sr & 1, abort_flag, lane)) goto teardown;
                tc_fence_after();
#pragma unroll 1
                for (int c = 0; c < C::N / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + c * 32, r);
                    tmem_wait_ld();
                    if (c == C::N / 32 - 1) {       // everything is in registers: the next accumulation may start
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(accempty);
                    }
#pragma unroll
                    for (int v = 0; v < 8; ++v)
                        red_add_f32x4(grow + c * 32 + v * 4, __uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                      __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                }
            }
            cur.next_unit(a, n_units, n_maps, n_tiles);
        }
    }

teardown:
    __syncwarp();
    if (*abort_flag) {
        if (tid == 0 && a.status) atomicExch(a.status, DEV_TIMEOUT);
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

int ts_sm_count()
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

template <bool COMP, bool CEN>
cudaError_t launch_ts(const TsParams &P, cudaStream_t st)
{
    using C = TsCfg<COMP>;
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(k_accum_ts<COMP, CEN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    const int n_units = 2 * P.a.Lt * P.a.Ht * P.a.n_splits;
    const int grid = n_units < ts_sm_count() ? n_units : ts_sm_count();
    k_accum_ts<COMP, CEN><<<grid, C::THREADS, C::SMEM_BYTES, st>>>(P);
    return cudaGetLastError();
}

}  // namespace

// d = 128, keys taken as stored (no rotary fold).  `comp`: hi + lo weighted operand.
cudaError_t launch_accum_ts(const AccumArgs &a, bool comp, const cb_kv_view *src, const cb_kv_view *tgt, cudaStream_t st)
{
    TsParams P;
    P.a = a;
    const int d = 128, TT = CB_TS_TT;
    if (!make_kv_tensor_map(&P.src_k, src->k, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                            src->stride_token, src->stride_layer, TT) ||
        !make_kv_tensor_map(&P.src_v, src->v, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                            src->stride_token, src->stride_layer, TT) ||
        !make_kv_tensor_map(&P.tgt_k, tgt->k, d, tgt->n_heads, tgt->n_tokens, tgt->n_layers, tgt->stride_head,
                            tgt->stride_token, tgt->stride_layer, TT) ||
        !make_kv_tensor_map(&P.tgt_v, tgt->v, d, tgt->n_heads, tgt->n_tokens, tgt->n_layers, tgt->stride_head,
                            tgt->stride_token, tgt->stride_layer, TT))
        return cudaErrorInvalidValue;
    // Tokens summed in tensor memory before a drain.  The tensor cores' fp32 accumulation loses about 1e-4 (relative,
    // on the all-positive sums of G) over 16,384 tokens; the compensated fold drains eight times as often, so that
    // its result stays an order of magnitude below the single-bf16 fold's error.
    P.drain_tiles = (comp ? 2048 : 16384) / TT;
    cudaError_t e;
    if (a.mu) e = comp ? launch_ts<true, true>(P, st) : launch_ts<false, true>(P, st);
    else e = comp ? launch_ts<true, false>(P, st) : launch_ts<false, false>(P, st);
    if (e == cudaSuccess) count_launch();
    return e;
}

}  // namespace cb
