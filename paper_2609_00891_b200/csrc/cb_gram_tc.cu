// Wide-regressor statistics on the tensor cores, 2 x 2 blocked (sm_100a): the full-head contrast (Section 3.1, Eq.
// "fullheadfeature") and the head-local support over k > 1 selected layers (Section 3.2).
//
// The feature of a group (full-head: one (component, target layer); head-local: one map) is F source heads of d
// channels.  G is F x F blocks of d x d, symmetric; C is F blocks per target head.  A thread block computes, per unit,
// the four d x d products of TWO weighted heads (rows) against TWO column heads:
//     G units (I, J), J <= I:  rows = feature heads 2I, 2I+1,  columns = feature heads 2J, 2J+1  (lower triangle,
//                              mirrored on write);
//     C units (I, hp):         rows = feature heads 2I, 2I+1,  columns = target heads 2hp, 2hp+1 (one target head for
//                              the head-local support).
// Four head tiles are staged per 64 tokens for four products, where the one-row-head kernel stages three for two: the
// kernel is bound by the L2-to-shared-memory feed, so the ratio is what counts, and the C units no longer carry a
// wasted diagonal product.
//
// Roles per block (persistent over units): warp 0 stages the two row heads (TMA); the last warp stages the two column
// heads and the token weights; 16 fold warps (8 per row head) replace the staged row heads by w .* rows IN PLACE (bf16)
// and keep the bias sums; warp 1 issues tcgen05.mma into two tensor-memory accumulators (all 512 columns at d = 128); 4 drain warps
// add a finished accumulator to G / C with fire-and-forget reductions (lower block triangle only; a mirror kernel
// fills the rest) (each output block has exactly one owner unit,
// and a thread's reductions to one address are performed in program order, so results are reproducible).
// Weighting in place leaves room for three stages of four 16 KB head tiles.  (Measured: the kernel is bound by the
// feed of those tiles into shared memory, ~7.6 TB/s over all SMs, plus ~640 cycles of synchronisation per tile: six
// stages of 32-token tiles were slower.)
// Every wait is bounded: if one runs out the block sets a flag, tears down and frees its tensor memory.
#include <cudaTypedefs.h>

#include "cb_internal.cuh"
#include "cb_ptx.cuh"
#include "cb_math.cuh"

namespace cb {

using namespace ptx;

template <int D>
struct GrCfg {
    static_assert(D == 128, "two 64-channel blocks per head make the M = 128 operand");
    static constexpr int TT = 64;
    static constexpr int NBX = D / 64;
    static constexpr int BLK = TT * 128;
    static constexpr int HEAD = NBX * BLK;                    // bytes of one staged head tile (16 KB)
    static constexpr int STAGE_BYTES = 4 * HEAD;              // [column head 0 | column head 1 | row head 0 | row head 1]
    static constexpr int NS = 3;
    static constexpr int N = 2 * D;                           // accumulator columns per row head
    static constexpr int TMEM_COLS = 2 * N;
    static constexpr int FOLD_WARPS = 16, GROUP_WARPS = 8, DRAIN_WARPS = 4;
    static constexpr int CPROD_WARP = 2 + FOLD_WARPS + DRAIN_WARPS;
    static constexpr int THREADS = (3 + FOLD_WARPS + DRAIN_WARPS) * 32;
    static constexpr int CC = D / 8;                          // 16-byte chunks per head row
    static constexpr int RG = GROUP_WARPS * 32 / CC;          // row groups of one fold group
    static constexpr int RPT = TT / RG;
    static constexpr int RED_STRIDE = 2 * D + 4;              // per fold warp: row-head sums [D], column-head sums [D], s_w
    static constexpr size_t SMEM_BYTES = 1024 + (size_t)NS * STAGE_BYTES + FOLD_WARPS * RED_STRIDE * 4 + NS * TT * 4 + 256;
    static_assert(RG % 8 == 0 && TT % RG == 0, "fold layout");
};

struct GrParams {
    CUtensorMap src_k, src_v, tgt_k, tgt_v;
    AccumArgs a;
    FullHeadArgs f;
    int sub_tiles;                // token tiles summed in tensor memory between two drains
    int FP, HPn, NGU, NCU;        // head pairs of the feature, target-head pairs, G and C blocks per group
};

// One unit, decoded once per unit by every role.
struct GrUnit {
    int u;
    int comp, l, h;               // h: target head of the map (head-local) or 0
    int group;
    int is_c;                     // C unit
    int diag;                     // G unit with I == J: the row heads are the column heads, staged once
    int I;
    int fa[2], va[2];             // row heads (feature index) and whether the second exists
    int fb[2], vb[2];             // column heads: feature index (G units) or target head (C units)
    int nb;                       // column heads staged (2, or 1 for the single target head of a head-local map)
    int own_sa, own_sy, own_sw;   // which bias entries this unit owns
    int la[2], ha[2], lb[2], hb[2];   // (layer, head) to load for rows / columns
    __device__ __forceinline__ void decode(const GrParams &P, int unit)
    {
        u = unit;
        const AccumArgs &a = P.a;
        const FullHeadArgs &f = P.f;
        // Unit order: block fastest, then group.  The blocks of a group read the same few heads and thread blocks
        // take consecutive units at about the same pace, so most tiles are served from L2.  Head-local groups are
        // ordered target layer fastest: neighbouring layers select almost the same source layers.
        const int per = P.NGU + P.NCU;
        const int v = u % per;
        const int gidx = u / per;
        int src_h = 0;
        if (f.per_head) {
            comp = gidx / (a.Lt * a.Ht);
            h = (gidx / a.Lt) % a.Ht;
            l = gidx % a.Lt;
            group = (comp * a.Lt + l) * a.Ht + h;
            src_h = f.src_head[h];
        } else {
            group = gidx;
            comp = group / a.Lt;
            l = group % a.Lt;
            h = 0;
        }
        auto feat_layer = [&](int ft) { return f.layer_sets[l * f.k + (f.per_head ? ft : ft / f.Hs)]; };
        auto feat_head = [&](int ft) { return f.per_head ? src_h : ft % f.Hs; };
        int J = 0, hp = 0;
        if (v < P.NGU) {
            is_c = 0;
            I = 0;
            while ((I + 1) * (I + 2) / 2 <= v) ++I;
            J = v - I * (I + 1) / 2;
        } else {
            is_c = 1;
            const int vc = v - P.NGU;
            I = vc / P.HPn;
            hp = vc % P.HPn;
        }
        fa[0] = 2 * I;
        va[0] = 1;
        va[1] = (2 * I + 1 < f.F) ? 1 : 0;
        fa[1] = va[1] ? 2 * I + 1 : 2 * I;
#pragma unroll
        for (int q = 0; q < 2; ++q) { la[q] = feat_layer(fa[q]); ha[q] = feat_head(fa[q]); }
        if (!is_c) {
            fb[0] = 2 * J;
            vb[0] = 1;
            vb[1] = (2 * J + 1 < f.F) ? 1 : 0;
            fb[1] = vb[1] ? 2 * J + 1 : 2 * J;
            nb = 2;
            diag = (I == J);
#pragma unroll
            for (int q = 0; q < 2; ++q) { lb[q] = feat_layer(fb[q]); hb[q] = feat_head(fb[q]); }
            own_sa = own_sy = own_sw = 0;
        } else {
            const int NH = f.per_head ? 1 : a.Ht;
            fb[0] = f.per_head ? h : 2 * hp;
            vb[0] = 1;
            vb[1] = (!f.per_head && 2 * hp + 1 < NH) ? 1 : 0;
            fb[1] = vb[1] ? 2 * hp + 1 : fb[0];
            nb = f.per_head ? 1 : 2;
            diag = 0;
#pragma unroll
            for (int q = 0; q < 2; ++q) { lb[q] = l; hb[q] = fb[q]; }
            own_sa = (hp == 0);
            own_sy = (I == 0);
            own_sw = (I == 0 && hp == 0);
        }
    }
    __device__ __forceinline__ const float *weights(const AccumArgs &a) const
    {
        return (comp ? a.w_v : a.w_k) + (long long)l * a.w_sl + (long long)h * a.w_sh;
    }
};


template <int D>
__global__ void __launch_bounds__(GrCfg<D>::THREADS, 1) k_gram2_tc(const __grid_constant__ GrParams P)
{
    using C = GrCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *stg = smem;                                          // [NS][STAGE_BYTES]
    float *red = reinterpret_cast<float *>(stg + (size_t)C::NS * C::STAGE_BYTES);
    float *wst = red + C::FOLD_WARPS * C::RED_STRIDE;             // [NS][TT]
    uint64_t *bars = reinterpret_cast<uint64_t *>(wst + C::NS * C::TT);
    uint64_t *full = bars;                  // [NS] row heads (1 arrival + bytes), column heads (1 + bytes), weights (32 lanes)
    uint64_t *empty = full + C::NS;         // [NS] MMA done with the stage
    uint64_t *afull = empty + C::NS;        // [NS] row heads weighted in place (every fold warp)
    uint64_t *accfull = afull + C::NS;      // [1]
    uint64_t *accempty = accfull + 1;       // [1]  (4 drain warps)
    uint64_t *redfull = accempty + 1;       // [1]
    uint64_t *reddone = redfull + 1;        // [1]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(reddone + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const AccumArgs &a = P.a;
    const FullHeadArgs &f = P.f;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_groups = 2 * a.Lt * (f.per_head ? a.Ht : 1);
    const int n_units = n_groups * (P.NGU + P.NCU);
    const int n_tiles = (a.n_tokens + C::TT - 1) / C::TT;
    const size_t PF = (size_t)f.PF;

    if (tid == 0) {
        for (int i = 0; i < C::NS; ++i) { mbar_init(&full[i], 2 + 32); mbar_init(&empty[i], 1); mbar_init(&afull[i], C::FOLD_WARPS); }
        mbar_init(accfull, 1);
        mbar_init(accempty, C::DRAIN_WARPS);
        mbar_init(redfull, C::FOLD_WARPS);
        mbar_init(reddone, C::FOLD_WARPS);
        abort_flag[0] = 0;
        abort_flag[1] = (int)P.a.poll_limit;
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
        // ================================ row-head producer (one thread) ================================
        if (lane == 0) {
            Ring<C::NS> st;
            GrUnit un;
            int itc = 0;
            for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
                un.decode(P, u);
                const CUtensorMap *map = un.comp ? &P.src_v : &P.src_k;
                const int nrow = 1 + un.va[1];
                for (int tile = 0; tile < n_tiles; ++tile, ++itc) {
                    if (!mbar_wait(&empty[st.idx], st.phase ^ 1, abort_flag)) goto teardown;
                    uint8_t *dst = stg + st.idx * C::STAGE_BYTES + 2 * C::HEAD;
                    if (un.diag) {
                        mbar_arrive(&full[st.idx]);              // the fold warps weight the column heads' tiles
                    } else {
                        mbar_arrive_expect_tx(&full[st.idx], nrow * C::HEAD);
                        tma_load_5d(dst, map, &full[st.idx], 0, tile * C::TT, 0, un.ha[0], un.la[0]);
                        if (un.va[1]) tma_load_5d(dst + C::HEAD, map, &full[st.idx], 0, tile * C::TT, 0, un.ha[1], un.la[1]);
                    }
                    st.next();
                }
            }
        }
    } else if (warp == C::CPROD_WARP) {
        // ================================ column-head + weights producer ================================
        Ring<C::NS> st;
        GrUnit un;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            un.decode(P, u);
            const CUtensorMap *map = un.is_c ? (un.comp ? &P.tgt_v : &P.tgt_k) : (un.comp ? &P.src_v : &P.src_k);
            const int ncol = (un.nb == 2 && un.vb[1]) ? 2 : 1;
            const float *w = un.weights(a);
            for (int tile = 0; tile < n_tiles; ++tile) {
                if (!mbar_wait_warp(&empty[st.idx], st.phase ^ 1, abort_flag, lane)) goto teardown;
                const int tok0 = tile * C::TT;
                if (lane == 0) {
                    uint8_t *dst = stg + st.idx * C::STAGE_BYTES;
                    mbar_arrive_expect_tx(&full[st.idx], ncol * C::HEAD);
                    tma_load_5d(dst, map, &full[st.idx], 0, tok0, 0, un.hb[0], un.lb[0]);
                    if (ncol == 2) tma_load_5d(dst + C::HEAD, map, &full[st.idx], 0, tok0, 0, un.hb[1], un.lb[1]);
                }
#pragma unroll
                for (int q = 0; q < C::TT / 32; ++q) {
                    const int r = lane + 32 * q;
                    const bool in = tok0 + r < a.n_tokens;
                    cp_async_4(&wst[st.idx * C::TT + r], w + (in ? tok0 + r : 0), in ? 4u : 0u);
                }
                cp_async_arrive_noinc(&full[st.idx]);
                st.next();
            }
        }
    } else if (warp == 1) {
        // ================================ MMA issuer (one thread) ================================
        if (lane == 0) {
            constexpr uint32_t idesc2 = umma_idesc_bf16(128, 2 * D, true, true);
            constexpr uint32_t idesc1 = umma_idesc_bf16(128, D, true, true);
            const uint64_t proto = umma_smem_desc_sw128(0, C::BLK, 1024);
            const uint32_t desc_hi = (uint32_t)(proto >> 32);
            const uint32_t b_lo0 = (uint32_t)proto | ((smem_u32(stg) & 0x3FFFFu) >> 4);
            Ring<C::NS> st;
            uint32_t sr = 0;
            int itm = 0;
            GrUnit un;
            for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
                un.decode(P, u);
                // a missing second column head (odd count) leaves stale bytes in its half of the stage: use N = D then
                const uint32_t idesc = (un.nb == 2 && un.vb[1]) ? idesc2 : idesc1;
                const int two_rows = un.va[1];
                for (int sr0 = 0; sr0 < n_tiles; sr0 += P.sub_tiles, ++sr) {
                    const int n_sub = min(n_tiles - sr0, P.sub_tiles);
                    if (!mbar_wait(accempty, (sr & 1) ^ 1, abort_flag)) goto teardown;
                    tc_fence_after();
                    uint32_t accum = 0;
                    for (int t = 0; t < n_sub; ++t, ++itm) {
                        if (!mbar_wait(&afull[st.idx], st.phase, abort_flag)) goto teardown;
                        tc_fence_after();
                        const uint32_t bl = b_lo0 + st.idx * (C::STAGE_BYTES >> 4);
                        const uint32_t al = bl + ((2 * C::HEAD) >> 4);                 // weighted row heads
#pragma unroll
                        for (int k = 0; k < C::TT / 16; ++k) {
                            const uint64_t bd = ((uint64_t)desc_hi << 32) | (bl + k * 128);
                            const uint32_t acc_flag = (k == 0) ? accum : 1u;
                            umma_bf16_ss(tmem_base, ((uint64_t)desc_hi << 32) | (al + k * 128), bd, idesc, acc_flag);
                            if (two_rows)
                                umma_bf16_ss(tmem_base + C::N, ((uint64_t)desc_hi << 32) | (al + (C::HEAD >> 4) + k * 128), bd, idesc, acc_flag);
                        }
                        accum = 1;
                        umma_commit(&empty[st.idx]);
                        st.next();
                    }
                    umma_commit(accfull);
                }
            }
        }
    } else if (warp < 2 + C::FOLD_WARPS) {
        // ================================ fold warps: group g weights row head g ================================
        const int fw = warp - 2;
        const int g = fw / C::GROUP_WARPS;
        const int gt = (fw % C::GROUP_WARPS) * 32 + lane;
        const int cc = gt % C::CC, rg = gt / C::CC;
        const int blk = cc >> 3, lc = cc & 7;
        const int off0 = blk * C::BLK + rg * 128 + ((lc ^ (rg & 7)) << 4);
        Ring<C::NS> st;
        uint32_t uc = 0;
        GrUnit un;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x, ++uc) {
            un.decode(P, u);
            const bool active = (g == 0) || un.va[1];                 // a missing second row head: nothing to weight
            const bool sum_rows = un.is_c && un.own_sa && active;
            const bool sum_cols = un.is_c && un.own_sy && ((g == 0) || (un.nb == 2 && un.vb[1]));
            uint64_t sa2[4], sb2[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) sa2[e] = sb2[e] = 0ull;
            float sw = 0.f;
            for (int t = 0; t < n_tiles; ++t) {
                if (!mbar_wait_warp(&full[st.idx], st.phase, abort_flag, lane)) goto teardown;
                const float *wsm = wst + st.idx * C::TT + rg;
                uint8_t *ah = stg + st.idx * C::STAGE_BYTES + (2 + g) * C::HEAD + off0;           // weighted row head g
                const uint8_t *cs = stg + st.idx * C::STAGE_BYTES + g * C::HEAD + off0;           // column head g
                const uint8_t *rs = un.diag ? cs : ah;      // rows to weight: staged in place, or the column head itself
                if (active) {
#pragma unroll
                    for (int i = 0; i < C::RPT; ++i) {
                        const int off = i * C::RG * 128;
                        const float wt = wsm[i * C::RG];
                        const uint64_t w2 = f2_pack(wt, wt);
                        const uint4 xv = *reinterpret_cast<const uint4 *>(rs + off);
                        const unsigned xu[4] = {xv.x, xv.y, xv.z, xv.w};
                        unsigned hw[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const uint64_t pr = f2_mul(w2, f2_from_bf16x2(xu[e]));
                            if (sum_rows) sa2[e] = f2_add(sa2[e], pr);
                            float p0, p1;
                            f2_unpack(pr, p0, p1);
                            hw[e] = pack_bf16x2(p0, p1);
                        }
                        *reinterpret_cast<uint4 *>(ah + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                        if (sum_cols) {
                            const uint4 yv = *reinterpret_cast<const uint4 *>(cs + off);
                            const unsigned yu[4] = {yv.x, yv.y, yv.z, yv.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) sb2[e] = f2_fma(w2, f2_from_bf16x2(yu[e]), sb2[e]);
                        }
                        if (cc == 0 && g == 0) sw += wt;
                    }
                } else if (sum_cols) {
#pragma unroll
                    for (int i = 0; i < C::RPT; ++i) {
                        const int off = i * C::RG * 128;
                        const float wt = wsm[i * C::RG];
                        const uint64_t w2 = f2_pack(wt, wt);
                        const uint4 yv = *reinterpret_cast<const uint4 *>(cs + off);
                        const unsigned yu[4] = {yv.x, yv.y, yv.z, yv.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) sb2[e] = f2_fma(w2, f2_from_bf16x2(yu[e]), sb2[e]);
                    }
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&afull[st.idx]);
                st.next();
            }
            // ---- bias entries (C units only): lanes holding the same channels add up, fixed-order sum over the
            //      group's warps, then one owner thread per entry adds to G / C ----
            if (un.is_c) {
                float sa[8], sb[8];
#pragma unroll
                for (int e = 0; e < 4; ++e) { f2_unpack(sa2[e], sa[2 * e], sa[2 * e + 1]); f2_unpack(sb2[e], sb[2 * e], sb[2 * e + 1]); }
                if (C::CC == 16) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        sa[e] += __shfl_xor_sync(0xffffffffu, sa[e], 16);
                        sb[e] += __shfl_xor_sync(0xffffffffu, sb[e], 16);
                    }
                    sw += __shfl_xor_sync(0xffffffffu, sw, 16);
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        sa[e] += __shfl_xor_sync(0xffffffffu, sa[e], 8);
                        sb[e] += __shfl_xor_sync(0xffffffffu, sb[e], 8);
                        sa[e] += __shfl_xor_sync(0xffffffffu, sa[e], 16);
                        sb[e] += __shfl_xor_sync(0xffffffffu, sb[e], 16);
                    }
                    sw += __shfl_xor_sync(0xffffffffu, sw, 8);
                    sw += __shfl_xor_sync(0xffffffffu, sw, 16);
                }
                if (!mbar_wait_warp(reddone, (uc & 1) ^ 1, abort_flag, lane)) goto teardown;
                float *rw = red + fw * C::RED_STRIDE;
                if (lane < C::CC) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) { rw[cc * 8 + e] = sa[e]; rw[D + cc * 8 + e] = sb[e]; }
                    if (cc == 0) rw[2 * D] = sw;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(redfull);
                if (!mbar_wait_warp(redfull, uc & 1, abort_flag, lane)) goto teardown;
                float *Gg = f.G + (size_t)un.group * PF * PF;
                // group g's 256 threads own the entries of row head g and column head g
                for (int v = gt; v < 2 * D + 1; v += C::GROUP_WARPS * 32) {
                    float sum = 0.f;
#pragma unroll
                    for (int q = 0; q < C::GROUP_WARPS; ++q) sum += red[(g * C::GROUP_WARPS + q) * C::RED_STRIDE + v];
                    if (v < D) {
                        if (un.own_sa && active) {
                            atomicAdd(&Gg[(PF - 1) * PF + (size_t)un.fa[g] * D + v], sum);     // bias row; the column is mirrored
                        }
                    } else if (v < 2 * D) {
                        if (un.own_sy && (g == 0 || (un.nb == 2 && un.vb[1]))) {
                            const size_t oc = f.per_head ? (size_t)un.group : (size_t)un.group * a.Ht + un.fb[g];
                            atomicAdd(&f.C[(oc * PF + (PF - 1)) * D + (v - D)], sum);
                        }
                    } else if (un.own_sw && g == 0) {
                        atomicAdd(&Gg[(PF - 1) * PF + (PF - 1)], sum);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(reddone);
            } else {
                // keep the two reduction barriers in step with the unit count
                if (!mbar_wait_warp(reddone, (uc & 1) ^ 1, abort_flag, lane)) goto teardown;
                if (lane == 0) mbar_arrive(redfull);
                if (!mbar_wait_warp(redfull, uc & 1, abort_flag, lane)) goto teardown;
                if (lane == 0) mbar_arrive(reddone);
            }
        }
    } else {
        // ================================ drain warps ================================
        const int q = warp & 3;
        const int row = q * 32 + lane;          // channel of the row head
        uint32_t sr = 0;
        GrUnit un;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            un.decode(P, u);
            float *Gg = f.G + (size_t)un.group * PF * PF;
            const int ncolh = (un.nb == 2 && un.vb[1]) ? 2 : 1;
            for (int sr0 = 0; sr0 < n_tiles; sr0 += P.sub_tiles, ++sr) {
                if (!mbar_wait_warp(accfull, sr & 1, abort_flag, lane, true, 4, 512)) goto teardown;
                tc_fence_after();
                if (row < D) {
                    for (int ra = 0; ra < 1 + un.va[1]; ++ra) {
                        const size_t ri = (size_t)un.fa[ra] * D + row;
#pragma unroll 1
                        for (int c = 0; c < ncolh * D / 16; ++c) {
                            uint32_t r[16];
                            tmem_ld_32x16(tmem_base + ((uint32_t)(q * 32) << 16) + ra * C::N + c * 16, r);
                            tmem_wait_ld();
                            const int part = (c * 16) / D, c0 = (c * 16) % D;
                            if (!un.is_c) {
                                const int j = un.fb[part], i = un.fa[ra];
                                if (j <= i) {                      // block row i, block column j <= i; the mirror kernel fills the rest
                                    float *dst = Gg + ri * PF + (size_t)j * D + c0;
#pragma unroll
                                    for (int e = 0; e < 16; ++e) atomicAdd(dst + e, __uint_as_float(r[e]));
                                }
                            } else {
                                const size_t oc = f.per_head ? (size_t)un.group : (size_t)un.group * a.Ht + un.fb[part];
                                float *dst = f.C + (oc * PF + ri) * D + c0;
#pragma unroll
                                for (int e = 0; e < 16; ++e) atomicAdd(dst + e, __uint_as_float(r[e]));
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(accempty);
            }
        }
    }

teardown:
    __syncwarp();
    if (*abort_flag) {
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

// G[c][r] = G[r][c] for r > c, per group; 32 x 32 tiles through shared memory so that both sides are coalesced.
__global__ void k_mirror_lower(float *__restrict__ G, int pf)
{
    if (blockIdx.y > blockIdx.x) return;                    // tile (row block x, column block y) with x >= y
    __shared__ float t[32][33];
    float *Gg = G + (size_t)blockIdx.z * pf * pf;
    const int r0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    for (int i = threadIdx.y; i < 32; i += 8) {
        const int r = r0 + i, c = c0 + threadIdx.x;
        t[i][threadIdx.x] = (r < pf && c < pf) ? Gg[(size_t)r * pf + c] : 0.f;
    }
    __syncthreads();
    for (int i = threadIdx.y; i < 32; i += 8) {
        const int c = c0 + i, r = r0 + threadIdx.x;         // writes G[c][r], r fastest
        if (r < pf && c < pf && r > c) Gg[(size_t)c * pf + r] = t[threadIdx.x][i];
    }
}

template <int D>
static cudaError_t launch_gr(const GrParams &P, int n_units, cudaStream_t st)
{
    using C = GrCfg<D>;
    static bool attr[MAX_DEVICES] = {};
    {
        cudaError_t e = opt_in_smem(k_gram2_tc<D>, (size_t)((int)C::SMEM_BYTES), attr);
        if (e != cudaSuccess) return e;
    }
    const int grid = n_units < device_sm_count() ? n_units : device_sm_count();
    k_gram2_tc<D><<<grid, C::THREADS, C::SMEM_BYTES, st>>>(P);
    return cudaGetLastError();
}

cudaError_t launch_gram2_tc(const AccumArgs &a, const FullHeadArgs &f, int d, const cb_kv_view *src, const cb_kv_view *tgt,
                            cudaStream_t st)
{
    GrParams P;
    P.a = a;
    P.f = f;
    const int TT = 64;
    if (!make_kv_tensor_map(&P.src_k, src->k, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                            src->stride_token, src->stride_layer, TT) ||
        !make_kv_tensor_map(&P.src_v, src->v, d, src->n_heads, src->n_tokens, src->n_layers, src->stride_head,
                            src->stride_token, src->stride_layer, TT) ||
        !make_kv_tensor_map(&P.tgt_k, tgt->k, d, tgt->n_heads, tgt->n_tokens, tgt->n_layers, tgt->stride_head,
                            tgt->stride_token, tgt->stride_layer, TT) ||
        !make_kv_tensor_map(&P.tgt_v, tgt->v, d, tgt->n_heads, tgt->n_tokens, tgt->n_layers, tgt->stride_head,
                            tgt->stride_token, tgt->stride_layer, TT))
        return cudaErrorInvalidValue;
    // The tensor-core accumulator truncates: at most 32,768 tokens are summed in tensor memory between drains (mean
    // relative drift of an all-positive sum ~2e-4 there), in equal parts.  A drain stalls the MMA thread here (both
    // accumulators belong to the unit), so fewer, longer parts than in the head-local k = 1 kernel.
    const int n_tiles = (a.n_tokens + TT - 1) / TT;
    const int cap = 32768 / TT;
    const int parts = (n_tiles + cap - 1) / cap;
    P.sub_tiles = (n_tiles + parts - 1) / (parts > 0 ? parts : 1);
    if (P.sub_tiles < 1) P.sub_tiles = 1;
    P.FP = (f.F + 1) / 2;
    const int NH = f.per_head ? 1 : a.Ht;
    P.HPn = (NH + 1) / 2;
    P.NGU = P.FP * (P.FP + 1) / 2;
    P.NCU = P.FP * P.HPn;
    const int n_groups = 2 * a.Lt * (f.per_head ? a.Ht : 1);
    const int n_units = n_groups * (P.NGU + P.NCU);
    if (d != 128) return cudaErrorInvalidValue;          // the caller routes other widths to the one-row-head kernel
    cudaError_t e = launch_gr<128>(P, n_units, st);
    if (e != cudaSuccess) return e;
    count_launch();
    // upper triangle <- lower triangle (the units only add to block rows >= block columns and to the bias row)
    const int pf = f.PF;
    dim3 grid((pf + 31) / 32, (pf + 31) / 32, n_groups);
    k_mirror_lower<<<grid, dim3(32, 8), 0, st>>>(f.G, pf);
    e = cudaGetLastError();
    if (e == cudaSuccess) count_launch();
    return e;
}

}  // namespace cb
