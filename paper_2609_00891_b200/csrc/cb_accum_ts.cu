// Head-local weighted statistics with the weighted operand in TENSOR MEMORY and the bias sum s_y on the tensor
// cores; plain, compensated, centred (two-pass) and rotary-boundary variants.  Written for 128-wide heads; a 64-wide
// head runs as a 128-wide one whose upper 64-channel block lies outside the tensor (the tile copies deliver it as
// zeros), and only the results of the real channels are written out.
//
// Same contraction as the shared-memory kernel (D[d][2d] = (w .* X)^T [X | Y] over tokens plus the bias sums), same
// units, slots and summation order of the splits.  What differs is where the first MMA operand lives: the fold warps
// write A = bf16(w x) straight into tensor memory (lane = channel, two tokens per 32-bit column) and the MMA reads it
// from there.  Per 64 tokens that saves the 16 KB shared-memory write of the weighted tile and its 16 KB read by
// the tensor cores and the shared-memory space of the operand buffers.  On full launches the board runs into its
// power limit (the SM clock measured inside the kernel falls to about 1.43 GHz, while each part of the kernel alone
// runs at 1.8 - 1.96 GHz): what counts is the energy per token, and most of what is left to save is instructions.
//
//   warp 0       X tile producer (TMA); warp 14: Y tile + token weights producer
//   warps 2..9   fold: a warp owns the channel quarter (warp % 4) that its tensor-memory lanes cover and one half of
//                the tile's tokens.  ldmatrix (8x8, transposed) delivers for thread i the pair (token 2j, 2j+1) of
//                channel i/4, which is exactly the register layout of the 16-lane x 128-bit tensor-memory store; the
//                swizzled tile is read without a transposition in registers.  s_x = sum w x falls out of the fold
//                (one packed add per two elements).  Each warp also writes the bf16 images w_hi, w_lo of 1/8 of the
//                tile's weights into a small K-major operand "wb" (16 rows per 64 tokens: w_hi, w_lo, zeros).
//   warp 1       MMA issuer, per 16 tokens:  D    += A [X | Y]   (A from tensor memory, N = 256)
//                                            D_sy += Y^T wb      (Y tile as the MN-major first operand, N = 16: the
//                                                                 w_hi and w_lo columns give s_y = sum_t w_t y_t
//                                                                 to 2^-17; products of bf16 are exact in fp32)
//                The small MMA replaces eight warps that summed w y on the ALUs (~600 warp instructions per 64
//                tokens, 0.4 ms of a 4.4 ms launch) at a cost of 0.15 ms.  Measured alternatives: s_x from a second
//                small MMA (A from tensor memory times a ones column) costs 0.08 ms alone but 0.25 ms beside the
//                s_y one (the tensor pipe is then 80 % busy at the capped clock); the packed add in the fold costs
//                0.07 ms.
//   warps 10..13 drain: tensor memory -> registers -> vector reductions onto the unit's slot (one writer per slot
//                and launch: the result does not depend on timing)
// Tensor memory: columns 0..255 the accumulator, 256..447 a ring of three weighted operands, 448..463 D_sy.
// One accumulator: the MMA waits while a unit's result is read out (about 1 % of a unit).
// Every wait is bounded: if one runs out the block sets the context's status word and tears down.
#include <cudaTypedefs.h>

#include "cb_internal.cuh"
#include "cb_ptx.cuh"
#include "cb_math.cuh"
#include "cb_rope.cuh"

namespace cb {

using namespace ptx;

namespace {

template <bool COMP>
struct TsCfg {
    static constexpr int D = 128;
    static constexpr int TT = COMP ? 64 : 128;   // tokens per tile (compensated: two operand images per tile)
    static constexpr int BLK = TT * 128;              // one 64-channel block of a tile: TT rows of 128 bytes
    static constexpr int STAGE_BYTES = 4 * BLK;       // [X blocks 0, 1 | Y blocks 0, 1]
    static constexpr int WB_BYTES = (TT / 64) * 2048; // per 64 tokens: 16 rows of 128 bytes (K-major, 128-byte swizzle)
    static constexpr int NS = TT == 128 ? 3 : 5;
    static constexpr int A_PARTS = COMP ? 2 : 1;
    static constexpr int A_PART_COLS = TT / 2;        // columns of one image of the weighted operand (two tokens per column)
    static constexpr int A_COLS = A_PART_COLS * A_PARTS;
    static constexpr int NA = 3;
    static constexpr int N = 2 * D;                   // accumulator columns
    static constexpr int A_COL0 = N;
    static constexpr int BIAS_COL = A_COL0 + NA * A_COLS;   // 16 columns of D_sy
    static constexpr int TMEM_COLS = 512;
    static constexpr int FOLD_WARPS = 8, DRAIN_WARPS = 4;
    static constexpr int YPROD_WARP = 2 + FOLD_WARPS + DRAIN_WARPS;
    static constexpr int THREADS = (YPROD_WARP + 1) * 32;
    static constexpr int TW = TT / FOLD_WARPS;        // tokens whose weights a fold warp converts
    static constexpr int RED_FLOATS = 2 * D + 16;     // s_x of the two token halves, partial s_w of the fold warps
    static constexpr size_t SMEM_BYTES = 1024 + (size_t)NS * (STAGE_BYTES + WB_BYTES) + RED_FLOATS * 4 + 2 * NS * TT * 4 + 256;
    static_assert(BIAS_COL + 16 <= TMEM_COLS, "tensor memory columns");
    static_assert(NA <= NS, "an operand buffer is released through its tile's stage barrier");
};

struct TsParams {
    CUtensorMap src_k, src_v, tgt_k, tgt_v;   // 5-D tiled maps: (64 channels, token, channel block, head, layer)
    AccumArgs a;
    int drain_tiles;                          // tiles accumulated in tensor memory between drains
    RopeDev rope;                             // ROPE kernels only
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

// CEN: two-pass centred construction: the weighted operand is w (x - mu_x) with the means of P.a.mu; s_y is not
// formed (the slot's entries stay zero); the slot's s_x entries become the column sums of the ROUNDED weighted
// operand (what the centred reduction needs for its exact correction).
// ROPE: key maps (comp = 0) are fitted in content coordinates (Section 3.1): before the fold proper, the fold warps
// rotate every source and target key row of the staged tile back by its position's angles IN PLACE (the tensor cores
// read the de-rotated rows as the second operand and for s_y); value maps take the ordinary path.
// NARROW: 64-wide heads (the upper 64-channel block of every tile is zero padding); the rotation then pairs channel i
// with i + 32 inside the first block.
template <bool COMP, bool CEN, bool ROPE, bool NARROW = false>
__global__ void __launch_bounds__(TsCfg<COMP>::THREADS, 1) k_accum_ts(const __grid_constant__ TsParams P)
{
    using C = TsCfg<COMP>;
    constexpr int D = C::D;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *xy = smem;                                       // [NS][STAGE_BYTES]
    uint8_t *wb = xy + (size_t)C::NS * C::STAGE_BYTES;        // [NS][WB_BYTES] rows 0, 1, 2 = w_hi, w_lo, ones
    float *redx = reinterpret_cast<float *>(wb + (size_t)C::NS * C::WB_BYTES);   // [2 token halves][D] partial s_x
    float *red = redx + 2 * D;                                // [FOLD_WARPS] partial s_w
    float *wst = red + 16;                                    // [NS][TT] token weights of the staged tile
    int *pst = reinterpret_cast<int *>(wst + C::NS * C::TT);  // [NS][TT] token positions (ROPE)
    uint64_t *bars = reinterpret_cast<uint64_t *>(pst + C::NS * C::TT);
    uint64_t *full = bars;                 // [NS] tile landed: X bytes (1 arrival), Y bytes (1), weights (32 lanes)
    uint64_t *empty = full + C::NS;        // [NS] stage free: MMA done (1) + every fold warp done
    uint64_t *afull = empty + C::NS;       // [NA] weighted operand written to tensor memory (every fold warp)
    uint64_t *accfull = afull + C::NA;     // [1]  accumulators complete (MMA)
    uint64_t *accempty = accfull + 1;      // [1]  accumulators read out (4 drain warps)
    uint64_t *redfull = accempty + 1;      // [1]  partial s_x, s_w of all fold warps written
    uint64_t *reddone = redfull + 1;       // [1]  partials consumed (fold warps 0..3)
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(reddone + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const AccumArgs &a = P.a;
    constexpr int dr = NARROW ? 64 : D;    // real head width: channels dr .. D - 1 are zero padding
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_maps = 2 * a.Lt * a.Ht;
    const int n_units = n_maps * a.n_splits;
    const int n_tiles = (a.n_tokens + C::TT - 1) / C::TT;

    if (tid == 0) {
        for (int i = 0; i < C::NS; ++i) { mbar_init(&full[i], 2 + 32); mbar_init(&empty[i], 1 + C::FOLD_WARPS); }
        for (int i = 0; i < C::NA; ++i) mbar_init(&afull[i], C::FOLD_WARPS);
        mbar_init(accfull, 1);
        mbar_init(accempty, C::DRAIN_WARPS);
        mbar_init(redfull, C::FOLD_WARPS);
        mbar_init(reddone, 4);
        abort_flag[0] = 0;
        abort_flag[1] = (int)P.a.poll_limit;
        mbar_fence_init();
        tma_prefetch_desc(&P.src_k); tma_prefetch_desc(&P.src_v);
        tma_prefetch_desc(&P.tgt_k); tma_prefetch_desc(&P.tgt_v);
    }
    if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
    // wb: rows 2..15 of every 16-row block stay zero; rows 0 and 1 are rewritten for every tile
    for (int i = tid; i < C::NS * C::WB_BYTES / 16; i += C::THREADS)
        *reinterpret_cast<uint4 *>(wb + (size_t)i * 16) = make_uint4(0u, 0u, 0u, 0u);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ================================ X producer (one thread) ================================
        if (lane == 0 && !a.starve) {       // starve (test hook): no source tile is ever requested
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
                    if (ROPE) cp_async_4(&pst[st.idx * C::TT + r], P.rope.pos + (in ? tok0 + r : 0), in ? 4u : 0u);
                }
                cp_async_arrive_noinc(&full[st.idx]);
                st.next();
                cur.advance(a, n_units, n_maps, n_tiles);
            } while (cur.u == u);
        }
    } else if (warp == 1) {
        // ================================ MMA issuer (one thread) ================================
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, C::N, false, true);     // A: tensor memory, B: MN-major
            constexpr uint32_t idesc_sy = umma_idesc_bf16(128, 16, true, false);    // A = Y tile: MN-major, B = wb
            const uint64_t proto = umma_smem_desc_sw128(0, C::BLK, 1024);
            const uint64_t proto_w = umma_smem_desc_sw128(0, 16, 1024);
            const uint32_t desc_hi = (uint32_t)(proto >> 32), w_hi32 = (uint32_t)(proto_w >> 32);
            const uint32_t b_lo0 = (uint32_t)proto | ((smem_u32(xy) & 0x3FFFFu) >> 4);
            const uint32_t w_lo0 = (uint32_t)proto_w | ((smem_u32(wb) & 0x3FFFFu) >> 4);
            const uint32_t d_sy = tmem_base + C::BIAS_COL;
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
                        const uint32_t wl = w_lo0 + st.idx * (C::WB_BYTES >> 4);
                        const uint32_t at = tmem_base + C::A_COL0 + ar.idx * C::A_COLS;
#pragma unroll
                        for (int k = 0; k < C::TT / 16; ++k) {
                            const uint32_t acc_k = (k == 0) ? accum : 1u;
                            const uint64_t bd = ((uint64_t)desc_hi << 32) | (bl + k * 128);   // 16 tokens = 2048 bytes
                            // wb: 64 tokens per 2048-byte block, 16 tokens = 32 bytes along the row
                            const uint64_t wd = ((uint64_t)w_hi32 << 32) | (wl + (k >> 2) * 128 + (k & 3) * 2);
                            umma_bf16_ts(tmem_base, at + k * 8, bd, idesc, acc_k);
                            if (COMP) umma_bf16_ts(tmem_base, at + C::A_PART_COLS + k * 8, bd, idesc, 1u);
                            if (!CEN) umma_bf16_ss(d_sy, ((uint64_t)desc_hi << 32) | (bl + ((2 * C::BLK) >> 4) + k * 128), wd, idesc_sy, acc_k);
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
        const int hf = fw >> 2;             // token half of the tile
        // ldmatrix row address of this lane: matrix j = lane / 8 is (8-channel chunk j & 1, token group j / 2), row
        // lane % 8 is a token; the 128-byte swizzle XORs the chunk index with the token's low three bits.
        const int lm_row = hf * (C::TT / 2) + 8 * (lane >> 4) + (lane & 7);
        uint32_t lm_off[2];
#pragma unroll
        for (int g = 0; g < 2; ++g)
            lm_off[g] = (q >> 1) * C::BLK + lm_row * 128 + (((4 * (q & 1) + 2 * g + ((lane >> 3) & 1)) ^ (lane & 7)) << 4);
        const uint32_t a_lane = tmem_base + ((uint32_t)(q * 32) << 16) + C::A_COL0 + hf * (C::TT / 4);
        // this lane's weight token (lanes below TW) and where its bf16 images go in wb (rows 0 and 1 of the block)
        const int wtok = fw * C::TW + (lane < C::TW ? lane : 0);
        // (64-token block, row n, 16-byte chunk (token / 8) XOR n, token % 8): rows 0 and 1
        const int wb_off0 = (wtok >> 6) * 2048 + (((wtok & 63) >> 3) << 4) + (wtok & 7) * 2;
        const int wb_off1 = (wtok >> 6) * 2048 + 128 + ((((wtok & 63) >> 3) ^ 1) << 4) + (wtok & 7) * 2;
        // ROPE: thread (rc, rr) rotates the frequencies 4 rc .. 4 rc + 3 (channels i and i + 64: the same place in the
        // two 64-channel blocks of a tile) of rows rr, rr + 16, ..  Along its rows the positions advance by 16 and from
        // tile to tile by TT, so (cos, sin) follow from the previous ones by one rotation with the thread's constants;
        // the polynomial is needed at the first tile of a unit, where positions break, and every 16th tile (drift).
        // Packed fp32 pairs: frequencies (4 rc, 4 rc + 1) and (4 rc + 2, 4 rc + 3).
        // A 64-wide head pairs channel i with i + 32, both in the tile's first 64-channel block (the second one is zero
        // padding): eight threads per row instead of sixteen, so a pass covers 32 rows and there are half as many
        // passes; in the swizzled row the partner chunk is the own one with address bit 6 flipped.
        constexpr bool narrow = NARROW;
        const int rc = narrow ? (tid - 64) & 7 : (tid - 64) & 15, rr = narrow ? (tid - 64) >> 3 : (tid - 64) >> 4;
        constexpr int rstep = narrow ? 32 : 16;                     // rows (and positions) between a thread's passes
        const int rp_off = rr * 128 + (((rc >> 1) ^ (rr & 7)) << 4) + (rc & 1) * 8;
        uint64_t rs16c[2] = {0ull, 0ull}, rs16s[2] = {0ull, 0ull}, rsTc[2] = {0ull, 0ull}, rsTs[2] = {0ull, 0ull};   // cos, sin of rstep theta, TT theta
        uint64_t seedc[2] = {0ull, 0ull}, seeds[2] = {0ull, 0ull};
        int seedpos = 0;
        if (ROPE) {
#pragma unroll
            for (int pp = 0; pp < 2; ++pp) {
                float c0, s0, c1, s1;
                rope_cs_poly(P.rope.f_src[rc * 4 + 2 * pp], rstep, c0, s0);
                rope_cs_poly(P.rope.f_src[rc * 4 + 2 * pp + 1], rstep, c1, s1);
                rs16c[pp] = f2_pack(c0, c1); rs16s[pp] = f2_pack(s0, s1);
                rope_cs_poly(P.rope.f_src[rc * 4 + 2 * pp], C::TT, c0, s0);
                rope_cs_poly(P.rope.f_src[rc * 4 + 2 * pp + 1], C::TT, c1, s1);
                rsTc[pp] = f2_pack(c0, c1); rsTs[pp] = f2_pack(s0, s1);
            }
        }
        Ring<C::NS> st, old;       // `old` trails `st` by NA tiles
        Ring<C::NA> ar;
        uint32_t it = 0, uc = 0;
        UnitIter cur;
        cur.start(a, n_units, n_maps, n_tiles);
        while (cur.valid(n_units)) {
            const int m = cur.m, split = cur.split, n_t = cur.tile1 - cur.tile;
            const bool rope_unit = ROPE && cur.comp == 0;
            uint64_t sx2[2][2];            // [16-channel group][chunk]: sums over this thread's token pairs
            uint64_t nmu2[2][2];
            float sw = 0.f;
#pragma unroll
            for (int g = 0; g < 2; ++g)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    sx2[g][c] = 0ull;
                    nmu2[g][c] = 0ull;
                    if (CEN && !rope_unit) {
                        const int ch = q * 32 + 16 * g + 8 * c + (lane >> 2);
                        const float mu = ch < dr ? __ldg(a.mu + (size_t)m * (2 * dr + 1) + ch) : 0.f;
                        nmu2[g][c] = f2_pack(-mu, -mu);
                    }
                }
            // CEN && ROPE, key maps: the rotation phase stores the de-rotated rows ALREADY CENTRED (source and target), so
            // that their rounding to bf16 is relative to the spread, not to the mean; the fold then has nothing to
            // subtract and the reduction nothing to correct.  Negated means of this thread's channels in the rotation's
            // layout: [source | target][pair pp] for the low and the high half of the head.
            uint64_t rmlo[2][2] = {{0ull, 0ull}, {0ull, 0ull}}, rmhi[2][2] = {{0ull, 0ull}, {0ull, 0ull}};
            if (CEN && rope_unit) {
                const float *mup = a.mu + (size_t)m * (2 * dr + 1);
#pragma unroll
                for (int xyi = 0; xyi < 2; ++xyi)
#pragma unroll
                    for (int pp = 0; pp < 2; ++pp) {
                        const float *b = mup + xyi * dr + rc * 4 + 2 * pp;
                        rmlo[xyi][pp] = f2_pack(-__ldg(b), -__ldg(b + 1));
                        rmhi[xyi][pp] = f2_pack(-__ldg(b + dr / 2), -__ldg(b + dr / 2 + 1));
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
                if (rope_unit) {
                    uint8_t *xt = xy + st.idx * C::STAGE_BYTES + rp_off;      // this thread's place in row rr of block 0
                    const int *pt = pst + st.idx * C::TT + rr;
                    const uint64_t neg1 = f2_pack(-1.f, -1.f);
                    constexpr int NI = C::TT / 16;
                    // positions of this thread's rows; `contig`: they advance by 16 from row to row (the common case:
                    // no sequence boundary inside the tile), decided once so that the row loop has no branches
                    constexpr int ni = narrow ? NI / 2 : NI;  // passes of this thread
                    int posv[NI];
#pragma unroll
                    for (int i = 0; i < NI; ++i) posv[i] = (i < ni) ? pt[rstep * i] : 0;
                    bool contig = true;
#pragma unroll
                    for (int i = 1; i < NI; ++i) contig = contig && (i >= ni || posv[i] == posv[0] + rstep * i);
                    uint64_t cc2[2], ss2[2];
                    if ((t == 0) || (posv[0] != seedpos + C::TT) || ((t & 15) == 0)) {
#pragma unroll
                        for (int pp = 0; pp < 2; ++pp) {
                            float c0, s0, c1, s1;
                            rope_cs_poly(P.rope.f_src[rc * 4 + 2 * pp], posv[0], c0, s0);
                            rope_cs_poly(P.rope.f_src[rc * 4 + 2 * pp + 1], posv[0], c1, s1);
                            cc2[pp] = f2_pack(c0, c1); ss2[pp] = f2_pack(s0, s1);
                        }
                    } else {
#pragma unroll
                        for (int pp = 0; pp < 2; ++pp) {            // angle += TT theta
                            cc2[pp] = f2_fma(seedc[pp], rsTc[pp], f2_mul(f2_mul(seeds[pp], rsTs[pp]), neg1));
                            ss2[pp] = f2_fma(seeds[pp], rsTc[pp], f2_mul(seedc[pp], rsTs[pp]));
                        }
                    }
                    seedc[0] = cc2[0]; seedc[1] = cc2[1]; seeds[0] = ss2[0]; seeds[1] = ss2[1]; seedpos = posv[0];
                    // rows rr + 16 i of the source tile, then of the target tile, turned back by (cc2, ss2) / (yc2, ys2)
                    auto rotate_rows = [&](int i, const uint64_t (&xc)[2], const uint64_t (&xs)[2], const uint64_t (&yc)[2],
                                           const uint64_t (&ys)[2]) {
#pragma unroll
                        for (int xyi = 0; xyi < 2; ++xyi) {
                            uint8_t *lo = xt + xyi * 2 * C::BLK + i * (rstep * 128);
                            uint8_t *hi = narrow ? reinterpret_cast<uint8_t *>(reinterpret_cast<uintptr_t>(lo) ^ 64) : lo + C::BLK;
                            const uint2 vl = *reinterpret_cast<const uint2 *>(lo), vh = *reinterpret_cast<const uint2 *>(hi);
                            const unsigned ul[2] = {vl.x, vl.y}, uh[2] = {vh.x, vh.y};
                            unsigned ol[2], oh[2];
#pragma unroll
                            for (int pp = 0; pp < 2; ++pp) {          // rotation by -phi
                                const uint64_t c2 = xyi ? yc[pp] : xc[pp], s2 = xyi ? ys[pp] : xs[pp];
                                const uint64_t l2 = f2_from_bf16x2(ul[pp]), h2 = f2_from_bf16x2(uh[pp]);
                                uint64_t nl = f2_fma(l2, c2, f2_mul(h2, s2));
                                uint64_t nh = f2_fma(h2, c2, f2_mul(f2_mul(l2, s2), neg1));
                                if (CEN) { nl = f2_add(nl, rmlo[xyi][pp]); nh = f2_add(nh, rmhi[xyi][pp]); }
                                float a0, a1;
                                f2_unpack(nl, a0, a1); ol[pp] = pack_bf16x2(a0, a1);
                                f2_unpack(nh, a0, a1); oh[pp] = pack_bf16x2(a0, a1);
                            }
                            *reinterpret_cast<uint2 *>(lo) = make_uint2(ol[0], ol[1]);
                            *reinterpret_cast<uint2 *>(hi) = make_uint2(oh[0], oh[1]);
                        }
                    };
                    auto target_angles = [&](int pos, uint64_t (&yc)[2], uint64_t (&ys)[2]) {
#pragma unroll
                        for (int pp = 0; pp < 2; ++pp) {
                            float c0, s0, c1, s1;
                            rope_cs_poly(P.rope.f_tgt[rc * 4 + 2 * pp], pos, c0, s0);
                            rope_cs_poly(P.rope.f_tgt[rc * 4 + 2 * pp + 1], pos, c1, s1);
                            yc[pp] = f2_pack(c0, c1); ys[pp] = f2_pack(s0, s1);
                        }
                    };
                    if (contig && P.rope.same) {
#pragma unroll
                        for (int i = 0; i < NI; ++i) {
                            if (i >= ni) break;
                            if (i > 0) {
#pragma unroll
                                for (int pp = 0; pp < 2; ++pp) {    // angle += 16 theta
                                    const uint64_t pc = cc2[pp], ps = ss2[pp];
                                    cc2[pp] = f2_fma(pc, rs16c[pp], f2_mul(f2_mul(ps, rs16s[pp]), neg1));
                                    ss2[pp] = f2_fma(ps, rs16c[pp], f2_mul(pc, rs16s[pp]));
                                }
                            }
                            rotate_rows(i, cc2, ss2, cc2, ss2);
                        }
                    } else {
#pragma unroll 1
                        for (int i = 0; i < ni; ++i) {
                            const int pos = pt[rstep * i];
                            if (i > 0) {
                                if (pos == pt[rstep * (i - 1)] + rstep) {
#pragma unroll
                                    for (int pp = 0; pp < 2; ++pp) {
                                        const uint64_t pc = cc2[pp], ps = ss2[pp];
                                        cc2[pp] = f2_fma(pc, rs16c[pp], f2_mul(f2_mul(ps, rs16s[pp]), neg1));
                                        ss2[pp] = f2_fma(ps, rs16c[pp], f2_mul(pc, rs16s[pp]));
                                    }
                                } else {
#pragma unroll
                                    for (int pp = 0; pp < 2; ++pp) {
                                        float c0, s0, c1, s1;
                                        rope_cs_poly(P.rope.f_src[rc * 4 + 2 * pp], pos, c0, s0);
                                        rope_cs_poly(P.rope.f_src[rc * 4 + 2 * pp + 1], pos, c1, s1);
                                        cc2[pp] = f2_pack(c0, c1); ss2[pp] = f2_pack(s0, s1);
                                    }
                                }
                            }
                            uint64_t yc2[2] = {cc2[0], cc2[1]}, ys2[2] = {ss2[0], ss2[1]};
                            if (!P.rope.same) target_angles(pos, yc2, ys2);
                            rotate_rows(i, cc2, ss2, yc2, ys2);
                        }
                    }
                    // every fold warp reads rows that other fold warps have just rewritten
                    asm volatile("bar.sync 1, %0;" ::"n"(C::FOLD_WARPS * 32) : "memory");
                }
                if (lane < C::TW) {
                    const float wv = wt[wtok];
                    const __nv_bfloat16 h = __float2bfloat16_rn(wv);
                    const __nv_bfloat16 l = __float2bfloat16_rn(wv - __bfloat162float(h));
                    uint8_t *dst = wb + st.idx * C::WB_BYTES;
                    *reinterpret_cast<__nv_bfloat16 *>(dst + wb_off0) = h;
                    *reinterpret_cast<__nv_bfloat16 *>(dst + wb_off1) = l;
                    sw += wv;
                }
                // 32 tokens of this warp's half at a time; token pairs of this lane: + 8 j + 2 (lane % 4) + {0, 1}
#pragma unroll
                for (int sub = 0; sub < C::TT / 64; ++sub) {
                    uint64_t w2[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        w2[j] = *reinterpret_cast<const uint64_t *>(wt + hf * (C::TT / 2) + sub * 32 + 8 * j + 2 * (lane & 3));
                    uint32_t r[2][2][4];
#pragma unroll
                    for (int g = 0; g < 2; ++g)
#pragma unroll
                        for (int tp = 0; tp < 2; ++tp) ldmatrix_x4_trans(stage_u32 + lm_off[g] + (sub * 32 + tp * 16) * 128, r[g][tp]);
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        uint32_t oh[8], ol[8];
#pragma unroll
                        for (int tp = 0; tp < 2; ++tp) {
#pragma unroll
                            for (int mi = 0; mi < 4; ++mi) {
                                uint64_t xf = f2_from_bf16x2(r[g][tp][mi]);
                                if (CEN) xf = f2_add(xf, nmu2[g][mi & 1]);                  // x - mu_x
                                const uint64_t pr = f2_mul(w2[2 * tp + (mi >> 1)], xf);      // w x for two tokens
                                if (!CEN) sx2[g][mi & 1] = f2_add(sx2[g][mi & 1], pr);
                                float p0, p1;
                                f2_unpack(pr, p0, p1);
                                const unsigned hw = pack_bf16x2(p0, p1);
                                oh[4 * tp + mi] = hw;
                                if (COMP) ol[4 * tp + mi] = pack_bf16x2(p0 - __uint_as_float(hw << 16), p1 - __uint_as_float(hw & 0xffff0000u));
                                if (CEN) {                                                  // sum of what the tensor cores will see
                                    sx2[g][mi & 1] = f2_add(sx2[g][mi & 1], f2_from_bf16x2(hw));
                                    if (COMP) sx2[g][mi & 1] = f2_add(sx2[g][mi & 1], f2_from_bf16x2(ol[4 * tp + mi]));
                                }
                            }
                        }
                        const uint32_t ta = a_lane + ((uint32_t)(16 * g) << 16) + ar.idx * C::A_COLS + sub * 16;
                        tmem_st_16x128_x4(ta, oh);
                        if (COMP) tmem_st_16x128_x4(ta + C::A_PART_COLS, ol);
                    }
                }
                tmem_wait_st();
                fence_async_smem();          // the wb rows (and rotated tiles) written above are read by the tensor cores
                tc_fence_before();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&afull[ar.idx]); mbar_arrive(&empty[st.idx]); }
                st.next();
                ar.next();
                ++it;
            }
            // ---- s_x and s_w of this unit: partial sums through shared memory, added in a fixed order ----
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) sw += __shfl_xor_sync(0xffffffffu, sw, o);
            if (!mbar_wait_warp(reddone, (uc & 1) ^ 1, abort_flag, lane)) goto teardown;
#pragma unroll
            for (int g = 0; g < 2; ++g)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    float lo, hi;
                    f2_unpack(sx2[g][c], lo, hi);
                    float v = lo + hi;
                    v += __shfl_xor_sync(0xffffffffu, v, 1);
                    v += __shfl_xor_sync(0xffffffffu, v, 2);
                    if ((lane & 3) == 0) redx[hf * D + q * 32 + 16 * g + 8 * c + (lane >> 2)] = v;
                }
            if (lane == 0) red[fw] = sw;
            __syncwarp();
            if (lane == 0) mbar_arrive(redfull);
            if (fw < 4) {
                if (!mbar_wait_warp(redfull, uc & 1, abort_flag, lane)) goto teardown;
                float *slot = a.slots + ((size_t)split * n_maps + m) * slot_floats(dr);
                const int v = fw * 32 + lane;
                if (v < dr) slot[slot_sx(dr) + v] += redx[v] + redx[D + v];
                if (v == 0) {
                    float sum = 0.f;
#pragma unroll
                    for (int k = 0; k < C::FOLD_WARPS; ++k) sum += red[k];
                    slot[slot_sw(dr)] += sum;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(reddone);
            }
            ++uc;
            cur.next_unit(a, n_units, n_maps, n_tiles);
        }
    } else {
        // ================================ drain warps ================================
        const int q = warp & 3;             // tensor-memory lane quarter this warp may access
        const int row = q * 32 + lane;      // row of D = channel of the weighted operand (D_sy: target channel)
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        uint32_t sr = 0;
        UnitIter cur;
        cur.start(a, n_units, n_maps, n_tiles);
        while (cur.valid(n_units)) {
            float *slot = a.slots + ((size_t)cur.split * n_maps + cur.m) * slot_floats(dr);
            float *grow = slot + (size_t)row * (2 * dr);             // row of the slot's [dr][2 dr] block
            for (int sr0 = cur.tile; sr0 < cur.tile1; sr0 += P.drain_tiles, ++sr) {
                if (!mbar_wait_warp(accfull, sr & 1, abort_flag, lane)) goto teardown;
                tc_fence_after();
                uint32_t b[16];
                tmem_ld_32x16(lane_base + C::BIAS_COL, b);
#pragma unroll 1
                for (int c = 0; c < C::N / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld_32x32(lane_base + c * 32, r);
                    tmem_wait_ld();
                    if (c == C::N / 32 - 1) {       // everything is in registers: the next accumulation may start
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(accempty);
                    }
                    // accumulator columns [0, D) are the source channels, [D, 2 D) the target channels; of each half
                    // the first dr columns are real, and so are the first dr rows
                    const int col = c * 32, half = col / D, cin = col % D;
                    if (row < dr && cin < dr) {
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            red_add_f32x4(grow + half * dr + cin + v * 4, __uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                          __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                    }
                }
                // D_sy columns 0 and 1: the w_hi and w_lo columns of wb
                if (!CEN && row < dr) atomicAdd(slot + slot_sy(dr) + row, __uint_as_float(b[0]) + __uint_as_float(b[1]));
            }
            cur.next_unit(a, n_units, n_maps, n_tiles);
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

template <bool COMP, bool CEN, bool ROPE = false, bool NARROW = false>
cudaError_t launch_ts(const TsParams &P, cudaStream_t st)
{
    using C = TsCfg<COMP>;
    static bool attr[MAX_DEVICES] = {};
    {
        cudaError_t e = opt_in_smem(k_accum_ts<COMP, CEN, ROPE, NARROW>, (size_t)((int)C::SMEM_BYTES), attr);
        if (e != cudaSuccess) return e;
    }
    const int n_units = 2 * P.a.Lt * P.a.Ht * P.a.n_splits;
    const int grid = n_units < device_sm_count() ? n_units : device_sm_count();
    k_accum_ts<COMP, CEN, ROPE, NARROW><<<grid, C::THREADS, C::SMEM_BYTES, st>>>(P);
    return cudaGetLastError();
}

}  // namespace

template <bool NARROW>
static cudaError_t launch_variant(const TsParams &P, bool comp, bool cen, bool rope, cudaStream_t st)
{
    if (rope) {
        if (cen) return comp ? launch_ts<true, true, true, NARROW>(P, st) : launch_ts<false, true, true, NARROW>(P, st);
        return comp ? launch_ts<true, false, true, NARROW>(P, st) : launch_ts<false, false, true, NARROW>(P, st);
    }
    if (cen) return comp ? launch_ts<true, true, false, NARROW>(P, st) : launch_ts<false, true, false, NARROW>(P, st);
    return comp ? launch_ts<true, false, false, NARROW>(P, st) : launch_ts<false, false, false, NARROW>(P, st);
}

// d = 128 or 64.  `comp`: hi + lo weighted operand.
cudaError_t launch_accum_ts(const AccumArgs &a, int d, bool comp, const cb_kv_view *src, const cb_kv_view *tgt, cudaStream_t st)
{
    TsParams P;
    P.a = a;
    const int TT = comp ? TsCfg<true>::TT : TsCfg<false>::TT;
    // the copy box always spans two 64-channel blocks: for d = 64 the second one is outside the tensor and arrives as zeros
    if (!make_kv_tensor_map(&P.src_k, src->k, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                            src->stride_token, src->stride_layer, TT, 2) ||
        !make_kv_tensor_map(&P.src_v, src->v, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                            src->stride_token, src->stride_layer, TT, 2) ||
        !make_kv_tensor_map(&P.tgt_k, tgt->k, d, tgt->n_heads, tgt->n_tokens, tgt->n_layers, tgt->stride_head,
                            tgt->stride_token, tgt->stride_layer, TT, 2) ||
        !make_kv_tensor_map(&P.tgt_v, tgt->v, d, tgt->n_heads, tgt->n_tokens, tgt->n_layers, tgt->stride_head,
                            tgt->stride_token, tgt->stride_layer, TT, 2))
        return cudaErrorInvalidValue;
    // Tokens summed in tensor memory before a drain.  The tensor cores' fp32 accumulation loses about 1e-4 (relative,
    // on the all-positive sums of G) over 16,384 tokens; the compensated fold drains eight times as often, so that
    // its result stays an order of magnitude below the single-bf16 fold's error.
    P.drain_tiles = (comp ? 2048 : 16384) / TT;
    cudaError_t e;
    P.rope = RopeDev{};
    if (a.rope_pos) {
        P.rope.pos = a.rope_pos;
        rope_frequencies(a.rope_base_src, d, P.rope.f_src);
        rope_frequencies(a.rope_base_tgt, d, P.rope.f_tgt);
        P.rope.same = (a.rope_base_src == a.rope_base_tgt) ? 1 : 0;
    }
    const bool rope = a.rope_pos != nullptr, cen = a.mu != nullptr;
    if (d == 64) e = launch_variant<true>(P, comp, cen, rope, st);
    else e = launch_variant<false>(P, comp, cen, rope, st);
    if (e == cudaSuccess) count_launch();
    return e;
}

}  // namespace cb
