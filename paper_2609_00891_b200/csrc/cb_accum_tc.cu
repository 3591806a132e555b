// Wide-regressor statistics with ONE row head per unit on the 5th-generation tensor cores (sm_100a), both MMA operands
// in shared memory: the full-head contrast and the head-local support over k > 1 layers under CB_FLAG_ONE_ROW_HEAD, and
// every wide-regressor call with 64-wide heads (the 2 x 2 blocked kernel of cb_gram_tc.cu serves d = 128).  Head-local
// k = 1 statistics run on the kernel that keeps the weighted operand in tensor memory (cb_accum_ts.cu); this file also
// holds the builder of the tiled tensor maps that all of these kernels use.
//
// A unit pairs one feature head A (its rows are weighted) with two heads [B1 | B2] (two feature heads for a block of G,
// or a feature head and a target head for a block of C):
//     D[d][2d] = (w .* A)^T [B1 | B2]          over tokens,
// plus, for C units, the bias sums s_a = sum w a, s_b = sum w b2, s_w = sum w kept on the ALUs.
//
// Per thread block (one per SM, persistent over its units):
//   warp 0      TMA producer for A and B1: tiles of TT tokens go straight from the strided cache layout to shared
//               memory (128-byte swizzle: one row = one token's 64 channels), NS stages deep.  The last warp does the
//               same for B2 and copies the tile's token weights.
//   fold warps  read the A tile, multiply each token row by its weight, round to bf16 (optionally hi+lo) into
//               the operand buffer in the same swizzled layout; accumulate the bias sums in registers.
//   warp 1      MMA issuer: tcgen05.mma, first operand = weighted tile (M = 128 channels, MN-major), second =
//               [B1 | B2] (N = 2d channels, MN-major), K = tokens, fp32 accumulator in tensor memory.
//   drain warps (4): when a unit's accumulator is complete, tensor memory -> registers -> added into G / C (every
//               entry has one owner unit); two accumulators let the next unit start meanwhile.
// Every wait is bounded: if one runs out the block sets the library's status word and tears down.
#include <cudaTypedefs.h>


#include "cb_internal.cuh"
#include "cb_ptx.cuh"
#include "cb_math.cuh"

namespace cb {

using namespace ptx;

template <int D, bool COMP>
struct TcCfg {
    static constexpr int TT = 64;                     // tokens per tile
    static constexpr int NBX = D / 64;                // 64-channel blocks per head
    static constexpr int BLK = TT * 128;              // bytes of one block: TT rows of 128 bytes
    // A stage holds the second MMA operand [B1 | B2] and, behind it, the head whose rows are weighted.
    static constexpr int STAGE_BYTES = 3 * NBX * BLK;
    static constexpr int AS_OFF = 2 * NBX * BLK;      // where the rows to be weighted start inside a stage
    static constexpr int A_BYTES = 2 * BLK;           // M = 128 always: two blocks (second stays zero for d = 64)
    static constexpr int NS = 3;                      // stages
    static constexpr int NA = 2;                    // weighted-operand buffers (hi, and lo when compensated)
    static constexpr int A_PARTS = COMP ? 2 : 1;
    static constexpr int N = 2 * D;                   // accumulator columns
    static constexpr int TMEM_COLS = 2 * N;           // two accumulators
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
                                         RED_FLOATS * 4 + NS * TT * 4 /*weights*/ + 256 /*barriers*/;
    static_assert(TT % RG == 0 && RPT >= 1, "fold layout");
    static_assert(TMEM_COLS == 256 || TMEM_COLS == 512, "tensor memory columns must be a power of two");
};

// Full-head contrast: per (component, target layer l) the feature is every KV head of k selected source
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
};

// Walks the tiles of this block's units in order: units u = blockIdx.x, += gridDim.x; unit -> (comp, l, G or C
// unit), all tiles.  The operands of a unit are decoded once per unit.
struct TileIter {
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
        {
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
        }
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


template <int D, bool COMP>
__global__ void __launch_bounds__(TcCfg<D, COMP>::THREADS, 1) k_accum_tc(const __grid_constant__ TcParams P)
{
    using C = TcCfg<D, COMP>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *xy = smem;                                       // [NS][STAGE_BYTES]
    uint8_t *ab = xy + (size_t)C::NS * C::STAGE_BYTES;        // [NA][hi A_BYTES (| lo A_BYTES)]
    float *red = reinterpret_cast<float *>(ab + (size_t)C::NA * C::A_PARTS * C::A_BYTES);
    float *wst = red + C::RED_FLOATS;                         // [NS][TT] token weights of the staged tile
    uint64_t *bars = reinterpret_cast<uint64_t *>(wst + C::NS * C::TT);
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
    const int n_units = 2 * a.Lt * (P.fh.per_head ? a.Ht : 1) * (P.fh.NG + P.fh.NC);
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
                    mbar_arrive_expect_tx(&full[st.idx], 2 * C::NBX * C::BLK);
                    tma_load_5d(xy + st.idx * C::STAGE_BYTES, map, &full[st.idx], 0, cur.tile * C::TT, 0, g, j);
                    tma_load_5d(xy + st.idx * C::STAGE_BYTES + C::AS_OFF, map, &full[st.idx], 0, cur.tile * C::TT, 0, ag, aj);
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
        Ring<C::NS> st, old;       // `old` trails `st` by NA tiles
        Ring<C::NA> ar;
        uint32_t it = 0, uc = 0;
        TileIter cur;
        cur.start(P, n_units, n_maps, n_tiles);
        while (cur.valid(n_units)) {
            const int n_t = cur.tile1 - cur.tile;
            uint64_t sx2[4], sy2[4];        // packed fp32 pairs: channels (2e, 2e+1) of this thread's chunk
#pragma unroll
            for (int e = 0; e < 4; ++e) sx2[e] = sy2[e] = 0ull;
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
                        const uint64_t xf = f2_from_bf16x2(xu[e]);
                        const uint64_t pr = f2_mul(w2, xf);                        // w * x for two channels
                        sx2[e] = f2_add(sx2[e], pr);
                        float p0, p1;
                        f2_unpack(pr, p0, p1);
                        hw[e] = pack_bf16x2(p0, p1);
                        if (COMP) lw[e] = pack_bf16x2(p0 - __uint_as_float(hw[e] << 16), p1 - __uint_as_float(hw[e] & 0xffff0000u));
                    }
                    *reinterpret_cast<uint4 *>(ah + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                    if (COMP) *reinterpret_cast<uint4 *>(ah + C::A_BYTES + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                    {
                        const uint4 yv = *reinterpret_cast<const uint4 *>(ys + off);
                        const unsigned yu[4] = {yv.x, yv.y, yv.z, yv.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) sy2[e] = f2_fma(w2, f2_from_bf16x2(yu[e]), sy2[e]);
                    }
                    if (cc == 0) sw += wt;
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
                    const int ch = cc * 8 + e;
                    rw[ch] = sx[e];
                    rw[D + ch] = sy[e];
                }
                if (cc == 0) rw[2 * D] = sw;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(redfull);
            if (!mbar_wait_warp(redfull, uc & 1, abort_flag, lane)) goto teardown;
            {
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
            for (int sr0 = cur.tile; sr0 < cur.tile1; sr0 += P.drain_tiles, ++sr) {
                const int acc = sr & 1;
                if (!mbar_wait_warp(&accfull[acc], (sr >> 1) & 1, abort_flag, lane, true, 4, 512)) goto teardown;
                tc_fence_after();
                {
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

template <int D, bool COMP>
static cudaError_t launch_tc(const TcParams &P, cudaStream_t st)
{
    using C = TcCfg<D, COMP>;
    static bool attr[MAX_DEVICES] = {};
    {
        cudaError_t e = opt_in_smem(k_accum_tc<D, COMP>, (size_t)((int)C::SMEM_BYTES), attr);
        if (e != cudaSuccess) return e;
    }
    const int n_units = 2 * P.a.Lt * (P.fh.per_head ? P.a.Ht : 1) * (P.fh.NG + P.fh.NC);
    const int grid = n_units < device_sm_count() ? n_units : device_sm_count();
    k_accum_tc<D, COMP><<<grid, C::THREADS, C::SMEM_BYTES, st>>>(P);
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

// Head-local statistics: both head widths run on the kernel that keeps the weighted operand in tensor memory
// (cb_accum_ts.cu; a 64-wide head runs there as a zero-padded 128-wide one).
cudaError_t launch_accum_tc(const AccumArgs &a, int d, const cb_kv_view *src, const cb_kv_view *tgt, cudaStream_t st)
{
    // Calls of fewer than 4,096 rows take the hi + lo weighted operand regardless of the flag: the single bf16
    // rounding averages out only like 1/sqrt(rows), such calls are bound by launch latency, not by the second MMA.
    const bool comp = a.compensated || a.n_tokens < 4096;
    return launch_accum_ts(a, d, comp, src, tgt, st);
}

cudaError_t launch_fullhead_tc(const AccumArgs &a, const FullHeadArgs &f, int d, const cb_kv_view *src, const cb_kv_view *tgt,
                               cudaStream_t st)
{
    TcParams P;
    P.a = a;
    P.fh = FhDev{f.G, f.C, f.layer_sets, f.gi, f.gq, f.src_head, f.F, f.k, f.Hs, f.PF, f.NG, f.NC, f.per_head};
    const int TT = 64;
    if (!fill_maps(P, d, src, tgt, TT)) return cudaErrorInvalidValue;
    P.drain_tiles = 16384 / TT;
    cudaError_t e = (d == 128) ? launch_tc<128, false>(P, st) : launch_tc<64, false>(P, st);
    if (e == cudaSuccess) count_launch();
    return e;
}

}  // namespace cb
