// Fused weighted-statistics accumulation on the 5th-generation tensor cores (sm_100a), both MMA operands in shared
// memory.  This kernel serves d = 64 and the one-row-head full-head variant; head-local calls with d = 128 go to
// the kernel that keeps the weighted operand in tensor memory (cb_accum_ts.cu).
//
// For one map (matched source head X, target head Y, token weights w) the statistics are the dense contraction
//     D[d][2d] = (w .* X)^T [X | Y]          over tokens,
// plus the bias sums s_x = sum w x, s_y = sum w y, s_w = sum w kept on the ALUs.
//
// Per thread block (one per SM, persistent over its units = (map, token split)):
//   warp 0      TMA producer for X: tiles of TT tokens go straight from the strided cache layout to shared memory
//               (128-byte swizzle: one row = one token's 64 channels), NS stages deep.  The last warp does the
//               same for Y and copies the tile's token weights.
//   fold warps  read the X tile, multiply each token row by its weight, round to bf16 (optionally hi+lo) into
//               the A buffer in the same swizzled layout; accumulate the bias sums in registers.
//   warp 1      MMA issuer: tcgen05.mma, A = weighted tile (M = 128 channels, MN-major), B = [X | Y]
//               (N = 2d channels, MN-major), K = tokens, fp32 accumulator in tensor memory.
//   drain warps (4): when a unit's accumulator is complete, tensor memory -> registers -> read-modify-write of
//               the unit's fp32 partial slot; two accumulators let the next unit start meanwhile.
// Every wait is bounded: if one runs out the block sets the context's status word and tears down.
#include <cudaTypedefs.h>


#include "cb_internal.cuh"
#include "cb_ptx.cuh"
#include "cb_math.cuh"
#include "cb_rope.cuh"

namespace cb {

using namespace ptx;

template <int D, bool COMP, bool FH = false, bool ROPE = false>
struct TcCfg {
    static constexpr int TT = 64;                     // tokens per tile
    static constexpr int NBX = D / 64;                // 64-channel blocks per head
    static constexpr int BLK = TT * 128;              // bytes of one block: TT rows of 128 bytes
    // A stage holds the second MMA operand [B1 | B2] (head-local: B1 = X, B2 = Y).  The rows to be weighted come
    // from B1; the full-head variant (FH) weights a third head, staged behind B2.
    static constexpr int STAGE_BYTES = (FH ? 3 : 2) * NBX * BLK;
    static constexpr int AS_OFF = FH ? 2 * NBX * BLK : 0;   // where the rows to be weighted start inside a stage
    static constexpr int A_BYTES = 2 * BLK;           // M = 128 always: two blocks (second stays zero for d = 64)
    static constexpr int NS = FH ? 3 : 4;   // stages (measured: 3 stages 3 % slower, 5 stages 1 % slower than 4)
    static constexpr int NA = 2;                    // weighted-operand buffers (hi, and lo when compensated)
    static constexpr int A_PARTS = COMP ? 2 : 1;
    static constexpr int N = 2 * D;                   // accumulator columns
    static constexpr int TMEM_COLS = 2 * N;           // two accumulators
    // ROPE: at most 8 fold warps, so that each fold thread may hold the rotation state of its rows in registers
    // (the block's register file divided by its threads caps a thread at 80 registers with 16 fold warps)
    static constexpr int FOLD_WARPS = 8, DRAIN_WARPS = 4;   // measured: 16 fold warps 1.5 % slower, 4 warps 6 % slower
    static constexpr int YPROD_WARP = 2 + FOLD_WARPS + DRAIN_WARPS;   // second producer: target tiles + weights
    static constexpr int FOLD_THREADS = FOLD_WARPS * 32;
    static constexpr int THREADS = (3 + FOLD_WARPS + DRAIN_WARPS) * 32;
    static constexpr int CC = D / 8;                  // 16-byte chunk columns of a head row
    static constexpr int RG = FOLD_THREADS / CC;      // row groups
    static constexpr int RPT = TT / RG;               // rows per fold thread
    static constexpr int RED_STRIDE = 2 * D + 4;                 // per fold warp: s_x[D], s_y[D], s_w, pad
    static constexpr int RED_FLOATS = FOLD_WARPS * RED_STRIDE;      // cross-warp bias reduction buffer
    static constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)NS * STAGE_BYTES + (size_t)NA * A_PARTS * A_BYTES +
                                         RED_FLOATS * 4 + 2 * NS * TT * 4 /*weights, positions*/ + 256 /*barriers*/;
    static_assert(TT % RG == 0 && RPT >= 1, "fold layout");
    static_assert(TMEM_COLS == 256 || TMEM_COLS == 512, "tensor memory columns must be a power of two");
};

// Full-head contrast (FH): per (component, target layer l) the feature is every KV head of k selected source
// layers: F = k*Hs feature heads.  Units per (comp, l): NG "G units" (i, q), 2q <= i: rows of feature head i against
// feature heads 2q and 2q+1 (the lower triangle of G, mirrored on write), then F*Ht "C units" (i, h): feature head i
// against target head h.  Results are added straight into G / C.
// per_head = 1 is the head-local support over k > 1 selected layers (Section 3.2): one group per map (comp, l, h),
// F = k feature heads (layer S_l[f], source head a(h)), weights per (l, h), G [n_maps][PF][PF], C [n_maps][PF][d].
struct FhDev {
    float *G, *C;                 // full-head: [2][Lt][PF][PF], [2][Lt][Ht][PF][d]
    const int *layer_sets;        // device [Lt][k]
    const int *gi, *gq;           // device [NG]
    const int *src_head;          // device [Ht] (per_head only)
    int F, k, Hs, PF, NG, NC, per_head;
};

struct TcParams {
    CUtensorMap src_k, src_v, tgt_k, tgt_v;   // 5-D tiled maps: (64 channels, token, channel block, head, layer)
    AccumArgs a;
    FhDev fh;
    int drain_tiles;                          // tiles accumulated in tensor memory between drains
    RopeDev rope;                             // ROPE kernels only
};

// Walks the tiles of this block's units in order: units u = blockIdx.x, += gridDim.x.  Head-local: unit -> (map,
// split) -> tiles [tile0, tile1); full-head: unit -> (comp, l, G or C unit), all tiles.  Empty units are skipped.
// The operands of a unit are decoded once per unit.
template <bool FH>
struct TileIterT {
    int u, tile, tile1, m, split;
    int comp, l, h;                 // component, target layer, target head (C units / head-local)
    int a_layer, a_head;            // source head whose rows are weighted
    int b1_layer, b1_head;          // first half of the second operand (a source head)
    int b2_layer, b2_head, b2_tgt;  // second half: target head (b2_tgt) or source head
    int fi, fj;                     // full-head: feature head of the rows; first feature head of the columns, or -1
    int out_g, out_c;               // full-head: which G matrix / C block the unit adds to
    int wr_sa, wr_sb, wr_sw;        // full-head C units: which bias entries this unit owns
    __device__ __forceinline__ void start(const TcParams &P, int n_units, int n_maps, int n_tiles)
    {
        u = (int)blockIdx.x - (int)gridDim.x;
        tile = tile1 = 0;
        next_unit(P, n_units, n_maps, n_tiles);
    }
    __device__ __forceinline__ bool valid(int n_units) const { return u < n_units; }
    __device__ __forceinline__ void next_unit(const TcParams &P, int n_units, int n_maps, int n_tiles)
    {
        const AccumArgs &a = P.a;
        if (FH) {
            u += gridDim.x;
            if (u >= n_units) return;
            const FhDev &f = P.fh;
            const int per = f.NG + f.NC;
            const int group = u / per, v = u % per;
            int src_h = 0;                                  // per_head: the one source head of this map
            if (f.per_head) {
                comp = group / (a.Lt * a.Ht);
                l = (group / a.Ht) % a.Lt;
                h = group % a.Ht;
                src_h = f.src_head[h];
            } else {
                comp = group / a.Lt;
                l = group % a.Lt;
                h = 0;
            }
            m = u; split = 0; tile = 0; tile1 = n_tiles;
            // feature head f -> (source layer, source head)
            auto feat_layer = [&](int ft) { return f.layer_sets[l * f.k + (f.per_head ? ft : ft / f.Hs)]; };
            auto feat_head = [&](int ft) { return f.per_head ? src_h : ft % f.Hs; };
            if (v < f.NG) {
                fi = f.gi[v];
                fj = 2 * f.gq[v];
                const int fj2 = (fj + 1 < f.F) ? fj + 1 : fj;    // odd F: the last pair repeats its first head (not stored)
                b1_layer = feat_layer(fj);   b1_head = feat_head(fj);
                b2_layer = feat_layer(fj2);  b2_head = feat_head(fj2);
                b2_tgt = 0;
                wr_sa = wr_sb = wr_sw = 0;
            } else {
                const int vc = v - f.NG;
                fj = -1;
                if (f.per_head) { fi = vc; }
                else { fi = vc / a.Ht; h = vc % a.Ht; }
                b1_layer = feat_layer(fi);   b1_head = feat_head(fi);
                b2_layer = l; b2_head = h; b2_tgt = 1;
                wr_sa = f.per_head ? 1 : (h == 0);
                wr_sb = (fi == 0);
                wr_sw = (fi == 0) && (f.per_head || h == 0);
            }
            a_layer = feat_layer(fi);
            a_head = feat_head(fi);
            out_g = group;
            out_c = f.per_head ? group : group * a.Ht + h;
            return;
        }
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
        a_layer = b1_layer = a.src_layer[l];
        a_head = b1_head = a.src_head[h];
        b2_layer = l; b2_head = h; b2_tgt = 1;
        fi = fj = 0;
    }
    __device__ __forceinline__ void advance(const TcParams &P, int n_units, int n_maps, int n_tiles)
    {
        if (++tile >= tile1) next_unit(P, n_units, n_maps, n_tiles);
    }
    __device__ __forceinline__ const float *weights(const AccumArgs &a) const
    {
        return (comp ? a.w_v : a.w_k) + (long long)l * a.w_sl + (long long)h * a.w_sh;   // full-head passes w_sh = 0
    }
};


// ROPE: key maps (comp = 0) are fitted in content coordinates (Section 3.1): the fold warps rotate every source and
// target key row back by its position's angles IN PLACE in the staged tile (so the tensor cores read the de-rotated
// rows as the second operand too) before weighting; value maps take the ordinary path.
// CEN: two-pass centred construction: the weighted operand is w (x - mu_x) with the means of P.a.mu; the bias sums
// become the column sums of the ROUNDED weighted operand (what the reduction needs for its exact correction).
template <int D, bool COMP, bool FH, bool CEN, bool ROPE>
__global__ void __launch_bounds__(TcCfg<D, COMP, FH, ROPE>::THREADS, 1) k_accum_tc(const __grid_constant__ TcParams P)
{
    using C = TcCfg<D, COMP, FH, ROPE>;
    using TileIter = TileIterT<FH>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *xy = smem;                                       // [NS][STAGE_BYTES]
    uint8_t *ab = xy + (size_t)C::NS * C::STAGE_BYTES;        // [NA][hi A_BYTES (| lo A_BYTES)]
    float *red = reinterpret_cast<float *>(ab + (size_t)C::NA * C::A_PARTS * C::A_BYTES);
    float *wst = red + C::RED_FLOATS;                         // [NS][TT] token weights of the staged tile
    int *pst = reinterpret_cast<int *>(wst + C::NS * C::TT);  // [NS][TT] token positions (ROPE)
    uint64_t *bars = reinterpret_cast<uint64_t *>(pst + C::NS * C::TT);
    uint64_t *full = bars;                 // [NS] tile landed: X bytes (1 arrival), Y bytes (1), weights (32 lanes)
    uint64_t *empty = full + C::NS;        // [NS] stage free: MMA done (1) + every fold warp done
    uint64_t *afull = empty + C::NS;       // [NA] weighted operand written (every fold warp)
    uint64_t *accfull = afull + C::NA;     // [2]  accumulator complete (MMA)
    uint64_t *accempty = accfull + 2;      // [2]  accumulator drained (4 drain warps)
    uint64_t *redfull = accempty + 2;      // [1]  bias partials of all fold warps written
    uint64_t *reddone = redfull + 1;       // [1]  bias partials consumed
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(reddone + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const AccumArgs &a = P.a;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_maps = 2 * a.Lt * a.Ht;
    const int n_units = FH ? 2 * a.Lt * (P.fh.per_head ? a.Ht : 1) * (P.fh.NG + P.fh.NC) : n_maps * a.n_splits;
    const int n_tiles = (a.n_tokens + C::TT - 1) / C::TT;

    if (tid == 0) {
        for (int i = 0; i < C::NS; ++i) { mbar_init(&full[i], 2 + 32); mbar_init(&empty[i], 1 + C::FOLD_WARPS); }
        for (int i = 0; i < C::NA; ++i) mbar_init(&afull[i], C::FOLD_WARPS);
        for (int i = 0; i < 2; ++i) { mbar_init(&accfull[i], 1); mbar_init(&accempty[i], C::DRAIN_WARPS); }
        mbar_init(redfull, C::FOLD_WARPS);
        mbar_init(reddone, C::FOLD_WARPS);
        abort_flag[0] = 0;
        abort_flag[1] = (int)P.a.poll_limit;
        mbar_fence_init();
        tma_prefetch_desc(&P.src_k); tma_prefetch_desc(&P.src_v);
        tma_prefetch_desc(&P.tgt_k); tma_prefetch_desc(&P.tgt_v);
    }
    if (warp == 1) tmem_alloc(tmem_slot, C::TMEM_COLS);
    if (D == 64 && warp >= 2 && warp < 2 + C::FOLD_WARPS) {
        // rows 64..127 of the M = 128 operand never get data: clear the second block of every A buffer once
        const int ft = tid - 64;
        for (int i = ft; i < C::NA * C::A_PARTS * (C::BLK / 16); i += C::FOLD_THREADS) {
            const int buf = i / (C::BLK / 16), off = i % (C::BLK / 16);
            *reinterpret_cast<uint4 *>(ab + (size_t)buf * C::A_BYTES + C::BLK + off * 16) = make_uint4(0, 0, 0, 0);
        }
        fence_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Every role walks the same tile sequence (TileIter).  The per-tile paths of the single-thread roles are kept
    // to a handful of instructions: a lone thread issues one dependent instruction every several cycles, so every
    // extra instruction there is paid once per tile by the whole pipeline.
    if (warp == 0) {
        // ================================ X producer (one thread) ================================
        if (lane == 0) {
            TileIter cur;
            cur.start(P, n_units, n_maps, n_tiles);
            Ring<C::NS> st;
            uint32_t it = 0;
            while (cur.valid(n_units)) {
                const CUtensorMap *map = cur.comp ? &P.src_v : &P.src_k;
                const int g = cur.b1_head, j = cur.b1_layer, ag = cur.a_head, aj = cur.a_layer, u = cur.u;
                do {   // tiles of one unit
                    if (!mbar_wait(&empty[st.idx], st.phase ^ 1, abort_flag)) goto teardown;
                    mbar_arrive_expect_tx(&full[st.idx], (FH ? 2 : 1) * C::NBX * C::BLK);
                    tma_load_5d(xy + st.idx * C::STAGE_BYTES, map, &full[st.idx], 0, cur.tile * C::TT, 0, g, j);
                    if (FH) tma_load_5d(xy + st.idx * C::STAGE_BYTES + C::AS_OFF, map, &full[st.idx], 0, cur.tile * C::TT, 0, ag, aj);
                    st.next();
                    ++it;
                    cur.advance(P, n_units, n_maps, n_tiles);
                } while (cur.u == u);
            }
        }
    } else if (warp == C::YPROD_WARP) {
        // ================================ Y + weights producer ================================
        // Lane 0 issues the Y tile copy; all 32 lanes copy the tile's token weights with 4-byte asynchronous copies
        // (zero-filled past the last token, no alignment requirement) that arrive on the same barrier.
        TileIter cur;
        cur.start(P, n_units, n_maps, n_tiles);
        Ring<C::NS> st;
        uint32_t it = 0;
        while (cur.valid(n_units)) {
            const CUtensorMap *map = cur.b2_tgt ? (cur.comp ? &P.tgt_v : &P.tgt_k) : (cur.comp ? &P.src_v : &P.src_k);
            const int h = cur.b2_head, l = cur.b2_layer, u = cur.u;
            const float *w = cur.weights(a);
            do {
                if (!mbar_wait_warp(&empty[st.idx], st.phase ^ 1, abort_flag, lane)) goto teardown;
                const int tok0 = cur.tile * C::TT;
                if (lane == 0) {
                    mbar_arrive_expect_tx(&full[st.idx], C::NBX * C::BLK);
                    tma_load_5d(xy + st.idx * C::STAGE_BYTES + C::NBX * C::BLK, map, &full[st.idx], 0, tok0, 0, h, l);
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
                ++it;
                cur.advance(P, n_units, n_maps, n_tiles);
            } while (cur.u == u);
        }
    } else if (warp == 1) {
        // ================================ MMA issuer (one thread) ================================
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, C::N, true, true);
            // Operand descriptors differ only in their 14-bit start-address field: keep the constant upper word and
            // the lower words of stage 0 / buffer 0, and step them with 32-bit adds.
            const uint64_t proto = umma_smem_desc_sw128(0, C::BLK, 1024);
            const uint32_t desc_hi = (uint32_t)(proto >> 32);
            const uint32_t b_lo0 = (uint32_t)proto | ((smem_u32(xy) & 0x3FFFFu) >> 4);
            const uint32_t a_lo0 = (uint32_t)proto | ((smem_u32(ab) & 0x3FFFFu) >> 4);
            Ring<C::NS> st;
            Ring<C::NA> ar;
            uint32_t it = 0, sr = 0;
            TileIter cur;
            cur.start(P, n_units, n_maps, n_tiles);
            while (cur.valid(n_units)) {
                const int u = cur.u, tile1 = cur.tile1;
                for (int sr0 = cur.tile; sr0 < tile1; sr0 += P.drain_tiles, ++sr) {
                    const int n_sub = min(tile1 - sr0, P.drain_tiles);
                    const uint32_t acc = sr & 1;
                    if (!mbar_wait(&accempty[acc], ((sr >> 1) & 1) ^ 1, abort_flag)) goto teardown;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * C::N;
                    uint32_t accum = 0;
                    for (int t = 0; t < n_sub; ++t) {
                        // afull implies full: every fold warp saw the tile land before it wrote the weighted operand
                        if (!mbar_wait(&afull[ar.idx], ar.phase, abort_flag)) goto teardown;
                        tc_fence_after();
                        const uint32_t bl = b_lo0 + st.idx * (C::STAGE_BYTES >> 4);
                        const uint32_t al = a_lo0 + ar.idx * ((C::A_PARTS * C::A_BYTES) >> 4);
#pragma unroll
                        for (int k = 0; k < C::TT / 16; ++k) {
                            const uint64_t bd = ((uint64_t)desc_hi << 32) | (bl + k * 128);
                            umma_bf16_ss(d_tmem, ((uint64_t)desc_hi << 32) | (al + k * 128), bd, idesc, k == 0 ? accum : 1u);
                            if (COMP) umma_bf16_ss(d_tmem, ((uint64_t)desc_hi << 32) | (al + (C::A_BYTES >> 4) + k * 128), bd, idesc, 1u);
                        }
                        accum = 1;
                        umma_commit(&empty[st.idx]);     // frees the stage and (through it) the weighted-operand buffer
                        st.next();
                        ar.next();
                        ++it;
                    }
                    umma_commit(&accfull[acc]);
                }
                while (cur.valid(n_units) && cur.u == u) cur.next_unit(P, n_units, n_maps, n_tiles);
            }
        }
    } else if (warp < 2 + C::FOLD_WARPS) {
        // ================================ fold warps ================================
        const int ft = tid - 64;
        const int cc = ft % C::CC, rg = ft / C::CC;
        const int blk = cc >> 3, lc = cc & 7;
        static_assert(C::RG % 8 == 0, "row groups must preserve the swizzle phase");
        // byte offset of this thread's first 16-byte chunk inside a block; its other rows are RG rows further down
        const int off0 = blk * C::BLK + rg * 128 + ((lc ^ (rg & 7)) << 4);
        float sx[8], sy[8], sw = 0.f;
        // ROPE: this thread rotates half a chunk (4 frequencies) of rows rg, rg + RG, ..: channels 4 cc + e pair with
        // channels D/2 + 4 cc + e.  Same (cc, rg) decomposition as the ordinary fold, other channels.
        // Between consecutive tiles of a sequence every position advances by TT, so (cos, sin) of a (row, frequency)
        // follow from the previous tile's by one rotation with the thread's constants (cos, sin)(TT theta_i); the
        // special-function unit (slow: it is shared by the whole scheduler) is only used at the first tile of a unit,
        // where the positions do not advance by TT, and every 16th tile to bound the drift of the recurrence.
        // Packed fp32 pairs throughout: frequencies (4 cc, 4 cc + 1) and (4 cc + 2, 4 cc + 3).
        uint64_t stc2[2] = {0ull, 0ull}, sts2[2] = {0ull, 0ull}, nsts2[2] = {0ull, 0ull};
        uint64_t rc2[C::RPT][2], rs2[C::RPT][2];
        int rprev[C::RPT];
        int rp_lo = 0, rp_hi = 0;
        if (ROPE) {
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                float c0, s0, c1, s1;
                rope_cs_poly(P.rope.f_src[cc * 4 + 2 * p], C::TT, c0, s0);
                rope_cs_poly(P.rope.f_src[cc * 4 + 2 * p + 1], C::TT, c1, s1);
                stc2[p] = f2_pack(c0, c1);
                sts2[p] = f2_pack(s0, s1);
                nsts2[p] = f2_pack(-s0, -s1);
            }
#pragma unroll
            for (int i = 0; i < C::RPT; ++i) {
                rprev[i] = 0;
#pragma unroll
                for (int p = 0; p < 2; ++p) { rc2[i][p] = f2_pack(1.f, 1.f); rs2[i][p] = 0ull; }
            }
            const int lcr = cc >> 1, hb = (cc & 1) * 8, swz = rg & 7;
            rp_lo = rg * 128 + ((lcr ^ swz) << 4) + hb;
            rp_hi = (D == 128) ? C::BLK + rp_lo : rg * 128 + (((lcr + 4) ^ swz) << 4) + hb;
        }
        Ring<C::NS> st, old;       // `old` trails `st` by NA tiles
        Ring<C::NA> ar;
        uint32_t it = 0, uc = 0;
        TileIter cur;
        cur.start(P, n_units, n_maps, n_tiles);
        while (cur.valid(n_units)) {
            const int m = cur.m, split = cur.split, n_t = cur.tile1 - cur.tile;
            const bool rope_unit = ROPE && cur.comp == 0;
            uint64_t sx2[4], sy2[4];        // packed fp32 pairs: channels (2e, 2e+1) of this thread's chunk
            uint64_t nmu2[4];               // centred: minus the means of those channels
#pragma unroll
            for (int e = 0; e < 4; ++e) sx2[e] = sy2[e] = nmu2[e] = 0ull;
            if (CEN) {
                const float *mup = a.mu + (size_t)m * (2 * D + 1) + cc * 8;
#pragma unroll
                for (int e = 0; e < 4; ++e) nmu2[e] = f2_pack(-__ldg(mup + 2 * e), -__ldg(mup + 2 * e + 1));
            }
            sw = 0.f;
            for (int t = 0; t < n_t; ++t) {
                if (!mbar_wait_warp(&full[st.idx], st.phase, abort_flag, lane)) goto teardown;
                // the weighted-operand buffer was last used by tile it - NA; it is free once that tile's stage is free
                if (it >= (uint32_t)C::NA) {
                    if (!mbar_wait_warp(&empty[old.idx], old.phase, abort_flag, lane)) goto teardown;
                    old.next();
                }
                const float *wsm = wst + st.idx * C::TT + rg;
                const uint8_t *xs = xy + st.idx * C::STAGE_BYTES + C::AS_OFF + off0;          // rows to be weighted
                const uint8_t *ys = xy + st.idx * C::STAGE_BYTES + C::NBX * C::BLK + off0;    // B2: summed with the weights
                uint8_t *ah = ab + ar.idx * (C::A_PARTS * C::A_BYTES) + off0;
                if (rope_unit) {
                    uint8_t *xt = xy + st.idx * C::STAGE_BYTES;                       // X tile, rewritten in place
                    uint8_t *yt = xt + C::NBX * C::BLK;                               // Y tile, rewritten in place
                    uint8_t *at = ab + ar.idx * (C::A_PARTS * C::A_BYTES);
                    const int *psm = pst + st.idx * C::TT + rg;
#pragma unroll
                    for (int i = 0; i < C::RPT; ++i) {
                        const int off = i * C::RG * 128;
                        const float wt = wsm[i * C::RG];
                        const uint64_t w2 = f2_pack(wt, wt);
                        const int pos = psm[i * C::RG];
                        uint64_t cs2[2], sn2[2];
                        if (t == 0 || pos != rprev[i] + C::TT || (t & 15) == 0) {
#pragma unroll
                            for (int p = 0; p < 2; ++p) {
                                float c0, s0, c1, s1;
                                rope_cs_poly(P.rope.f_src[cc * 4 + 2 * p], pos, c0, s0);
                                rope_cs_poly(P.rope.f_src[cc * 4 + 2 * p + 1], pos, c1, s1);
                                cs2[p] = f2_pack(c0, c1);
                                sn2[p] = f2_pack(s0, s1);
                            }
                        } else {
#pragma unroll
                            for (int p = 0; p < 2; ++p) {                              // angle += TT theta
                                cs2[p] = f2_fma(rc2[i][p], stc2[p], f2_mul(rs2[i][p], nsts2[p]));
                                sn2[p] = f2_fma(rs2[i][p], stc2[p], f2_mul(rc2[i][p], sts2[p]));
                            }
                        }
                        rprev[i] = pos;
#pragma unroll
                        for (int p = 0; p < 2; ++p) { rc2[i][p] = cs2[p]; rs2[i][p] = sn2[p]; }
                        const uint64_t neg1 = f2_pack(-1.f, -1.f);
                        uint64_t nsn2[2] = {f2_mul(sn2[0], neg1), f2_mul(sn2[1], neg1)};
                        {
                            const uint2 vl = *reinterpret_cast<const uint2 *>(xt + rp_lo + off);
                            const uint2 vh = *reinterpret_cast<const uint2 *>(xt + rp_hi + off);
                            const unsigned ul[2] = {vl.x, vl.y}, uh[2] = {vh.x, vh.y};
                            unsigned xl[2], xh[2], al[2], ah2[2], bl[2], bh[2];
#pragma unroll
                            for (int p = 0; p < 2; ++p) {                              // rotation by -phi
                                const uint64_t lo2 = f2_from_bf16x2(ul[p]), hi2 = f2_from_bf16x2(uh[p]);
                                const uint64_t nl2 = f2_fma(lo2, cs2[p], f2_mul(hi2, sn2[p]));
                                const uint64_t nh2 = f2_fma(hi2, cs2[p], f2_mul(lo2, nsn2[p]));
                                const uint64_t pl2 = f2_mul(w2, nl2), ph2 = f2_mul(w2, nh2);
                                sx2[p] = f2_add(sx2[p], pl2);
                                sx2[2 + p] = f2_add(sx2[2 + p], ph2);
                                float a0, a1;
                                f2_unpack(nl2, a0, a1); xl[p] = pack_bf16x2(a0, a1);
                                f2_unpack(nh2, a0, a1); xh[p] = pack_bf16x2(a0, a1);
                                float q0, q1, r0, r1;
                                f2_unpack(pl2, q0, q1); al[p] = pack_bf16x2(q0, q1);
                                f2_unpack(ph2, r0, r1); ah2[p] = pack_bf16x2(r0, r1);
                                if (COMP) {
                                    bl[p] = pack_bf16x2(q0 - __uint_as_float(al[p] << 16), q1 - __uint_as_float(al[p] & 0xffff0000u));
                                    bh[p] = pack_bf16x2(r0 - __uint_as_float(ah2[p] << 16), r1 - __uint_as_float(ah2[p] & 0xffff0000u));
                                }
                            }
                            *reinterpret_cast<uint2 *>(xt + rp_lo + off) = make_uint2(xl[0], xl[1]);
                            *reinterpret_cast<uint2 *>(xt + rp_hi + off) = make_uint2(xh[0], xh[1]);
                            *reinterpret_cast<uint2 *>(at + rp_lo + off) = make_uint2(al[0], al[1]);
                            *reinterpret_cast<uint2 *>(at + rp_hi + off) = make_uint2(ah2[0], ah2[1]);
                            if (COMP) {
                                *reinterpret_cast<uint2 *>(at + C::A_BYTES + rp_lo + off) = make_uint2(bl[0], bl[1]);
                                *reinterpret_cast<uint2 *>(at + C::A_BYTES + rp_hi + off) = make_uint2(bh[0], bh[1]);
                            }
                        }
                        if (!P.rope.same) {
#pragma unroll
                            for (int p = 0; p < 2; ++p) {
                                float c0, s0, c1, s1;
                                rope_cs_poly(P.rope.f_tgt[cc * 4 + 2 * p], pos, c0, s0);
                                rope_cs_poly(P.rope.f_tgt[cc * 4 + 2 * p + 1], pos, c1, s1);
                                cs2[p] = f2_pack(c0, c1);
                                sn2[p] = f2_pack(s0, s1);
                                nsn2[p] = f2_pack(-s0, -s1);
                            }
                        }
                        {
                            const uint2 vl = *reinterpret_cast<const uint2 *>(yt + rp_lo + off);
                            const uint2 vh = *reinterpret_cast<const uint2 *>(yt + rp_hi + off);
                            const unsigned ul[2] = {vl.x, vl.y}, uh[2] = {vh.x, vh.y};
                            unsigned yl[2], yh[2];
#pragma unroll
                            for (int p = 0; p < 2; ++p) {
                                const uint64_t lo2 = f2_from_bf16x2(ul[p]), hi2 = f2_from_bf16x2(uh[p]);
                                const uint64_t nl2 = f2_fma(lo2, cs2[p], f2_mul(hi2, sn2[p]));
                                const uint64_t nh2 = f2_fma(hi2, cs2[p], f2_mul(lo2, nsn2[p]));
                                sy2[p] = f2_fma(w2, nl2, sy2[p]);
                                sy2[2 + p] = f2_fma(w2, nh2, sy2[2 + p]);
                                float a0, a1;
                                f2_unpack(nl2, a0, a1); yl[p] = pack_bf16x2(a0, a1);
                                f2_unpack(nh2, a0, a1); yh[p] = pack_bf16x2(a0, a1);
                            }
                            *reinterpret_cast<uint2 *>(yt + rp_lo + off) = make_uint2(yl[0], yl[1]);
                            *reinterpret_cast<uint2 *>(yt + rp_hi + off) = make_uint2(yh[0], yh[1]);
                        }
                        if (cc == 0) sw += wt;
                    }
                } else {
#pragma unroll
                for (int i = 0; i < C::RPT; ++i) {
                    const int off = i * C::RG * 128;
                    const float wt = wsm[i * C::RG];
                    const uint64_t w2 = f2_pack(wt, wt);
                    const uint4 xv = *reinterpret_cast<const uint4 *>(xs + off);
                    const unsigned xu[4] = {xv.x, xv.y, xv.z, xv.w};
                    unsigned hw[4], lw[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        uint64_t xf = f2_from_bf16x2(xu[e]);
                        if (CEN) xf = f2_add(xf, nmu2[e]);                         // x - mu_x
                        const uint64_t pr = f2_mul(w2, xf);                        // w * x for two channels
                        if (!CEN) sx2[e] = f2_add(sx2[e], pr);
                        float p0, p1;
                        f2_unpack(pr, p0, p1);
                        hw[e] = pack_bf16x2(p0, p1);
                        if (COMP) lw[e] = pack_bf16x2(p0 - __uint_as_float(hw[e] << 16), p1 - __uint_as_float(hw[e] & 0xffff0000u));
                        if (CEN) {                                                 // sum of what the tensor cores will see
                            sx2[e] = f2_add(sx2[e], f2_from_bf16x2(hw[e]));
                            if (COMP) sx2[e] = f2_add(sx2[e], f2_from_bf16x2(lw[e]));
                        }
                    }
                    *reinterpret_cast<uint4 *>(ah + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                    if (COMP) *reinterpret_cast<uint4 *>(ah + C::A_BYTES + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                    if (!CEN) {
                        const uint4 yv = *reinterpret_cast<const uint4 *>(ys + off);
                        const unsigned yu[4] = {yv.x, yv.y, yv.z, yv.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) sy2[e] = f2_fma(w2, f2_from_bf16x2(yu[e]), sy2[e]);
                    }
                    if (cc == 0) sw += wt;
                }
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&afull[ar.idx]); mbar_arrive(&empty[st.idx]); }
                st.next();
                ar.next();
                ++it;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) { f2_unpack(sx2[e], sx[2 * e], sx[2 * e + 1]); f2_unpack(sy2[e], sy[2 * e], sy[2 * e + 1]); }
            // ---- bias sums of this unit: lanes holding the same channels add up, then a fixed-order sum over the
            //      warps, then read-modify-write of the slot ----
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
            if (!mbar_wait_warp(reddone, (uc & 1) ^ 1, abort_flag, lane)) goto teardown;
            float *rw = red + fw * C::RED_STRIDE;
            if (lane < C::CC) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    // ordinary fold: channels 8 cc + e; rotated key units: 4 cc + e and D/2 + 4 cc + (e - 4)
                    const int ch = rope_unit ? ((e < 4) ? cc * 4 + e : D / 2 + cc * 4 + (e - 4)) : cc * 8 + e;
                    rw[ch] = sx[e];
                    rw[D + ch] = sy[e];
                }
                if (cc == 0) rw[2 * D] = sw;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(redfull);
            if (!mbar_wait_warp(redfull, uc & 1, abort_flag, lane)) goto teardown;
            if (FH) {
                // C units carry the bias entries (each entry has exactly one owner, see the unit decode).
                if (cur.fj < 0) {
                    const FhDev &f = P.fh;
                    const size_t PF = (size_t)f.PF;
                    float *Gg = f.G + (size_t)cur.out_g * PF * PF;
                    float *Cg = f.C + (size_t)cur.out_c * PF * D;
                    for (int v = ft; v < 2 * D + 1; v += C::FOLD_THREADS) {
                        float sum = 0.f;
#pragma unroll
                        for (int q = 0; q < C::FOLD_WARPS; ++q) sum += red[q * C::RED_STRIDE + v];
                        if (v < D) {
                            if (cur.wr_sa) {
                                Gg[((size_t)cur.fi * D + v) * PF + (PF - 1)] += sum;
                                Gg[(PF - 1) * PF + (size_t)cur.fi * D + v] += sum;
                            }
                        } else if (v < 2 * D) {
                            if (cur.wr_sb) Cg[(PF - 1) * D + (v - D)] += sum;
                        } else if (cur.wr_sw) {
                            Gg[(PF - 1) * PF + (PF - 1)] += sum;
                        }
                    }
                }
            } else {
                float *slot = a.slots + ((size_t)split * n_maps + m) * slot_floats(D);
                for (int v = ft; v < 2 * D + 1; v += C::FOLD_THREADS) {
                    float sum = 0.f;
#pragma unroll
                    for (int q = 0; q < C::FOLD_WARPS; ++q) sum += red[q * C::RED_STRIDE + v];
                    slot[slot_sx(D) + v] += sum;    // s_x, s_y, s_w are adjacent in the slot
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(reddone);
            ++uc;
            cur.next_unit(P, n_units, n_maps, n_tiles);
        }
    } else {
        // ================================ drain warps ================================
        const int q = warp & 3;             // tensor-memory lane quarter this warp may access
        const int row = q * 32 + lane;      // row of D = channel of the weighted operand
        uint32_t sr = 0;
        TileIter cur;
        cur.start(P, n_units, n_maps, n_tiles);
        while (cur.valid(n_units)) {
            float *slot = FH ? nullptr : a.slots + ((size_t)cur.split * n_maps + cur.m) * slot_floats(D);
            for (int sr0 = cur.tile; sr0 < cur.tile1; sr0 += P.drain_tiles, ++sr) {
                const int acc = sr & 1;
                if (!mbar_wait_warp(&accfull[acc], (sr >> 1) & 1, abort_flag, lane, true, 4, 512)) goto teardown;
                tc_fence_after();
                if (FH) {
                    if (row < D) {
                        const FhDev &f = P.fh;
                        const size_t PF = (size_t)f.PF;
                        float *Gg = f.G + (size_t)cur.out_g * PF * PF;
                        const size_t ri = (size_t)cur.fi * D + row;           // row of G / C this thread holds
#pragma unroll 1
                        for (int c = 0; c < C::N / 16; ++c) {
                            uint32_t r[16];
                            tmem_ld_32x16(tmem_base + ((uint32_t)(q * 32) << 16) + acc * C::N + c * 16, r);
                            tmem_wait_ld();
                            const int part = (c * 16) / D, c0 = (c * 16) % D;   // which half of [B1 | B2], first column
                            if (cur.fj >= 0) {
                                const int j = cur.fj + part;                    // feature head of these columns
                                if (j <= cur.fi && j < f.F) {
                                    float *dst = Gg + ri * PF + (size_t)j * D + c0;
#pragma unroll
                                    for (int e = 0; e < 16; ++e) dst[e] += __uint_as_float(r[e]);
                                    if (j < cur.fi) {                           // mirror into the upper triangle
                                        float *mir = Gg + ((size_t)j * D + c0) * PF + ri;
#pragma unroll
                                        for (int e = 0; e < 16; ++e) mir[(size_t)e * PF] += __uint_as_float(r[e]);
                                    }
                                }
                            } else if (part == 1) {
                                float *dst = f.C + ((size_t)cur.out_c * PF + ri) * D + c0;
#pragma unroll
                                for (int e = 0; e < 16; ++e) dst[e] += __uint_as_float(r[e]);
                            }
                        }
                    }
                } else if (row < D) {
                    float *grow = slot + (size_t)row * C::N;
#pragma unroll 1
                    for (int c = 0; c < C::N / 16; ++c) {
                        uint32_t r[16];
                        float4 g[4];
#pragma unroll
                        for (int v = 0; v < 4; ++v) g[v] = *reinterpret_cast<const float4 *>(grow + c * 16 + v * 4);
                        tmem_ld_32x16(tmem_base + ((uint32_t)(q * 32) << 16) + acc * C::N + c * 16, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            g[v].x += __uint_as_float(r[4 * v + 0]);
                            g[v].y += __uint_as_float(r[4 * v + 1]);
                            g[v].z += __uint_as_float(r[4 * v + 2]);
                            g[v].w += __uint_as_float(r[4 * v + 3]);
                            *reinterpret_cast<float4 *>(grow + c * 16 + v * 4) = g[v];
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&accempty[acc]);
            }
            cur.next_unit(P, n_units, n_maps, n_tiles);
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

// 5-D map over (64 channels, token, 64-channel block, head, layer).  One box = box_tokens tokens of one head of
// one layer, laid out in shared memory as [channel block][token][64 channels] with the 128-byte swizzle.
// box_cblocks: 64-channel blocks per box (0: all d / 64 of them; 1: one block, selected by the copy's third coordinate).
bool make_kv_tensor_map(CUtensorMap *map, const void *base, int d, int H, long long T, int L,
                        long long sh, long long st, long long sl, int box_tokens, int box_cblocks)
{
    PFN_cuTensorMapEncodeTiled_v12000 enc = encode_fn();
    if (!enc) return false;
    auto stride = [&](long long elems, long long size) -> cuuint64_t {
        return (size == 1 || elems == 0) ? (cuuint64_t)d * 2 : (cuuint64_t)elems * 2;   // size-1 dimension: any valid stride
    };
    cuuint64_t gdim[5] = {64, (cuuint64_t)T, (cuuint64_t)(d / 64), (cuuint64_t)H, (cuuint64_t)L};
    cuuint64_t gstr[4] = {stride(st, T), 128, stride(sh, H), stride(sl, L)};
    cuuint32_t box[5] = {64, (cuuint32_t)box_tokens, (cuuint32_t)(box_cblocks > 0 ? box_cblocks : d / 64), 1, 1}, estr[5] = {1, 1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(base), gdim, gstr, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <int D, bool COMP, bool FH = false, bool CEN = false, bool ROPE = false>
static cudaError_t launch_tc(const TcParams &P, cudaStream_t st)
{
    using C = TcCfg<D, COMP, FH, ROPE>;
    static bool attr[MAX_DEVICES] = {};
    {
        cudaError_t e = opt_in_smem(k_accum_tc<D, COMP, FH, CEN, ROPE>, (size_t)((int)C::SMEM_BYTES), attr);
        if (e != cudaSuccess) return e;
    }
    const int n_units = FH ? 2 * P.a.Lt * (P.fh.per_head ? P.a.Ht : 1) * (P.fh.NG + P.fh.NC) : 2 * P.a.Lt * P.a.Ht * P.a.n_splits;
    const int grid = n_units < device_sm_count() ? n_units : device_sm_count();
    k_accum_tc<D, COMP, FH, CEN, ROPE><<<grid, C::THREADS, C::SMEM_BYTES, st>>>(P);
    return cudaGetLastError();
}

static bool fill_maps(TcParams &P, int d, const cb_kv_view *src, const cb_kv_view *tgt, int TT)
{
    return make_kv_tensor_map(&P.src_k, src->k, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                              src->stride_token, src->stride_layer, TT) &&
           make_kv_tensor_map(&P.src_v, src->v, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                              src->stride_token, src->stride_layer, TT) &&
           make_kv_tensor_map(&P.tgt_k, tgt->k, d, tgt->n_heads, tgt->n_tokens, tgt->n_layers, tgt->stride_head,
                              tgt->stride_token, tgt->stride_layer, TT) &&
           make_kv_tensor_map(&P.tgt_v, tgt->v, d, tgt->n_heads, tgt->n_tokens, tgt->n_layers, tgt->stride_head,
                              tgt->stride_token, tgt->stride_layer, TT);
}

cudaError_t launch_accum_tc(const AccumArgs &a, int d, const cb_kv_view *src, const cb_kv_view *tgt, cudaStream_t st)
{
    // Calls of fewer than 4,096 rows take the hi + lo weighted operand regardless of the flag: the single bf16
    // rounding averages out only like 1/sqrt(rows), such calls are bound by launch latency, not by the second MMA.
    const bool comp = a.compensated || a.n_tokens < 4096;
    // d = 128: the kernel that keeps the weighted operand in tensor memory
    if (d == 128) return launch_accum_ts(a, comp, src, tgt, st);
    TcParams P;
    P.a = a;
    P.fh = FhDev{};
    P.rope = RopeDev{};
    if (a.rope_pos) {
        P.rope.pos = a.rope_pos;
        rope_frequencies(a.rope_base_src, d, P.rope.f_src);
        rope_frequencies(a.rope_base_tgt, d, P.rope.f_tgt);
        P.rope.same = (a.rope_base_src == a.rope_base_tgt) ? 1 : 0;
    }
    const int TT = 64;
    if (!fill_maps(P, d, src, tgt, TT)) return cudaErrorInvalidValue;
    cudaError_t e;
    // Tokens summed in tensor memory before a drain (the fp32 accumulation of the tensor cores loses about 1e-4 over
    // 16,384 tokens; the compensated fold drains eight times as often).
    P.drain_tiles = (comp ? 2048 : 16384) / TT;
    if (a.rope_pos) e = comp ? launch_tc<64, true, false, false, true>(P, st) : launch_tc<64, false, false, false, true>(P, st);
    else if (a.mu) e = comp ? launch_tc<64, true, false, true>(P, st) : launch_tc<64, false, false, true>(P, st);
    else e = comp ? launch_tc<64, true>(P, st) : launch_tc<64, false>(P, st);
    if (e == cudaSuccess) count_launch();
    return e;
}

cudaError_t launch_fullhead_tc(const AccumArgs &a, const FullHeadArgs &f, int d, const cb_kv_view *src, const cb_kv_view *tgt,
                               cudaStream_t st)
{
    TcParams P;
    P.a = a;
    P.fh = FhDev{f.G, f.C, f.layer_sets, f.gi, f.gq, f.src_head, f.F, f.k, f.Hs, f.PF, f.NG, f.NC, f.per_head};
    P.rope = RopeDev{};
    const int TT = 64;
    if (!fill_maps(P, d, src, tgt, TT)) return cudaErrorInvalidValue;
    P.drain_tiles = 16384 / TT;
    cudaError_t e = (d == 128) ? launch_tc<128, false, true>(P, st) : launch_tc<64, false, true>(P, st);
    if (e == cudaSuccess) count_launch();
    return e;
}

}  // namespace cb
