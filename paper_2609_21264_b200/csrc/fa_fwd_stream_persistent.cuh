// Persistent form of the stream kernel (fa_fwd_stream.cuh; read that file first: same roles, same TMEM map, same
// arithmetic): one CTA per SM walks a list of work items, one 128-row query tile each, so that a CTA's fixed
// cost (launch, set-up, first loads, epilogue drain: about 11 000 cycles against 1300-1450 per K/V tile) is paid
// once per SM instead of once per query tile, and the loads of the next item run under the last tiles and the
// epilogue of the current one.  Fixed-length batches without split-KV and without shared query tiles.
//
// Item list: the order of the one-item kernel's grid (L2-sized groups of heads, inside a group every head's last
// query tile first: longest items first under a causal mask).  CTA c starts with item c and draws every further item
// from a ticket counter in global memory, so the items in flight are always a window of consecutive list entries,
// as they are when the hardware hands out one-item CTAs.  (A fixed assignment, item n G + c or a snake over rounds,
// was measured first: the CTAs drift apart by their items' lengths, the window spreads over several L2 groups, and
// DRAM reads grew from 1.15 GB to 6.3 GB on B 1, H 128, S 8192 at 192/128.)  The thread that loads Q and K draws the
// tickets, one item ahead of the CTA's compute, and hands every item to the other roles through a small ring in
// shared memory (item_full / item_empty).
//
// What carries over from item to item:
//   * every mbarrier keeps running: a role counts the K/V tiles of all its items (tile j of an item whose
//     predecessors had T tiles is tile T + j of the CTA: it uses S/P buffer pair (T + j) & 1, for the
//     ((T + j) >> 1)-th time, and belongs to softmax warpgroup (T + j) & 1, so that the two warpgroups keep
//     alternating across items with odd numbers of tiles and an item's first tile goes to the warpgroup that did not
//     run the last tile of the item before), the ring positions of K and V, and the items it has finished;
//   * the O accumulator: the first PV product of an item (accumulate = 0) waits until the epilogue of the item before
//     has read O out of TMEM (o_read);
//   * the output is staged for its TMA store in a stage of the V ring (an O tile is exactly as large as a V tile): every
//     item takes one more ring position than it has V tiles, the one after its last V tile, which nothing is loaded
//     into and whose "empty" arrival comes from the storing thread instead of an MMA commit.  (The V ring, not the K
//     ring: with two stages of each at 192/128 the stage comes back only when the store has read it, and the next
//     item's second V tile is needed a softmax pass later than its second K tile.)  So the query tile's
//     space is free as soon as the item's last score MMA is complete (q_free, a commit), and the next item's Q and
//     first K/V tiles are loaded, and its first scores computed, under the last softmax passes, the last PV products
//     and the epilogue of the current item.
//   * the epilogue belongs to the correction warps, which have nothing else to do then (one thread per query row,
//     as for the rescale): they take the two warpgroups' partial row sums, wait for the item's last PV product, read O
//     out of TMEM, normalise, stage and store it.  The softmax warps publish their sums and go straight on to the next
//     item, whose first passes run under the last PV product and the epilogue of this one.
// Items without a visible key (more queries than keys under a causal mask) have no loads, no MMAs and no barrier
// traffic: the softmax warps write their zeros and -inf and every role moves on.
#pragma once

#include "fa_fwd_stream.cuh"

namespace fa {

struct StreamPersistShared {
    uint64_t q_full;         // loader -> score MMA: the item's query tile has landed
    uint64_t q_free;         // score MMA -> loader: the item's last score MMA is complete, the query tile's space is free
    uint64_t k_full[4], k_empty[4];
    uint64_t v_full[4], v_empty[4];
    uint64_t s_full[2], s_free[2], st_full[2], p_ready[2], p_free[2];      // as in StreamShared
    uint64_t o_final;        // PV MMA -> epilogue: the item's last PV product is complete
    uint64_t o_read;         // correction warps -> PV MMA: the epilogue has read O out of TMEM
    uint64_t l_ready;        // softmax warps -> correction warps: partial row sums (and the final u) published
    uint64_t state_read;     // correction warps -> softmax warps: the epilogue has read them
    uint64_t o_staged;       // correction warps -> storing thread
    uint64_t item_full[4];   // loader -> every other role: ring slot holds the index of the CTA's next item (-1: none)
    uint64_t item_empty[4];  // the 15 consumers (8 softmax warps, 4 correction warps, 2 MMA threads, V loader) -> loader
    int item_ring[4];
    float alpha[2][kTileM];
    float mref[kTileM];
    float lsum[2][kTileM];
    uint32_t tmem_base;
    uint32_t abort_flag;
};

template <int DQK, int DV>
constexpr int stream_persist_smem_bytes() {
    return StreamCfg<DQK, DV>::kTileBytes + static_cast<int>(sizeof(StreamPersistShared));
}

// Registers per thread after the per-role reallocation (512 threads start with 128 each): the roles that walk the item
// list carry a few more values than in the one-item kernel.  256 x 184 + 128 x 72 + 128 x 72 = 65536.
constexpr int kSpRegsSoftmax = 184, kSpRegsCorrection = 72, kSpRegsOther = 72;

// One work item: a query tile of a head.
struct StreamItem {
    int q_tile, hq, b, kvh, i0, n_kv;
};

template <int DQK, int DV>
__global__ void __launch_bounds__(512, 1)
fa_fwd_stream_persistent_kernel(const __grid_constant__ CUtensorMap tm_q,
                                const __grid_constant__ CUtensorMap tm_k,
                                const __grid_constant__ CUtensorMap tm_v,
                                const __grid_constant__ CUtensorMap tm_o,
                                const FwdParams p) {
    using Cfg = StreamCfg<DQK, DV>;
    using namespace ptx;
    constexpr int NK = Cfg::kKStages;
    constexpr int NV = Cfg::kVStages;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    StreamPersistShared& sh = *reinterpret_cast<StreamPersistShared*>(smem_raw + Cfg::kTileBytes);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    grid_launch_dependents();

    const uint32_t smem_base = smem_addr(smem_raw);
    if ((smem_base & 1023u) != 0u) {          // uniform over the CTA; nothing has been set up yet
        grid_dependency_wait();
        if (tid == 0 && p.status) {
            volatile uint32_t* sw = p.status;
            sw[1] = kSiteSmemAlign;
            sw[0] = 3u;                       // FA_ERR_CUDA
            __threadfence_system();
        }
        return;
    }
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + Cfg::kQBytes;
    const uint32_t sV = sK + NK * Cfg::kKBytes;

    const int n_bh = p.B * p.Hq;
    const int n_items = p.n_q_tiles * n_bh;
    const int G = static_cast<int>(gridDim.x);
    const int cta = static_cast<int>(blockIdx.x);
    const int Sq = p.Sq, Sk = p.Sk;
    const int off = Sk - Sq;
    auto decode = [&](int item, StreamItem& it) {
        const int per_group = p.n_q_tiles * p.heads_per_group;
        const int group = item / per_group;
        const int bh0 = group * p.heads_per_group;
        const int group_size = (n_bh - bh0 < p.heads_per_group) ? (n_bh - bh0) : p.heads_per_group;
        const int local = item - group * per_group;
        it.q_tile = p.n_q_tiles - 1 - local / group_size;
        const int bh = bh0 + local % group_size;
        it.hq = bh % p.Hq;
        it.b = bh / p.Hq;
        it.kvh = it.hq / (p.Hq / p.Hkv);
        it.i0 = it.q_tile * kTileM;
        it.n_kv = kv_tiles_for_q_tile(it.i0, kTileM, Sq, Sk, p.causal);
    };

    // ---------------------------------------------------------------- setup
    if (tid == 0) {
        sh.abort_flag = 0;
        mbar_init(smem_addr(&sh.q_full), 1);
        mbar_init(smem_addr(&sh.q_free), 1);
        mbar_init(smem_addr(&sh.o_final), 1);
        mbar_init(smem_addr(&sh.o_read), 4);
        mbar_init(smem_addr(&sh.l_ready), 8);
        mbar_init(smem_addr(&sh.state_read), 4);
        mbar_init(smem_addr(&sh.o_staged), 4);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_addr(&sh.s_full[i]), 1);
            mbar_init(smem_addr(&sh.s_free[i]), 4);
            mbar_init(smem_addr(&sh.st_full[i]), 4);
            mbar_init(smem_addr(&sh.p_ready[i]), 8);
            mbar_init(smem_addr(&sh.p_free[i]), 1);
        }
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            mbar_init(smem_addr(&sh.item_full[s]), 1);
            mbar_init(smem_addr(&sh.item_empty[s]), 15);
            mbar_init(smem_addr(&sh.k_full[s]), 1);
            mbar_init(smem_addr(&sh.k_empty[s]), 1);
            mbar_init(smem_addr(&sh.v_full[s]), 1);
            mbar_init(smem_addr(&sh.v_empty[s]), 1);
        }
        fence_mbar_init();
    }
    if (warp == 12) {
        tmem_alloc(smem_addr(&sh.tmem_base), Cfg::kTmemCols);
        tmem_relinquish_alloc_permit();
    }
    if (warp == 14 && lane == 0) {
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
        prefetch_tensormap(&tm_o);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    grid_dependency_wait();

    const uint32_t tmem_base = sh.tmem_base;
    WaitCtx wctx{&sh.abort_flag, p.status, p.wait_limit_ns};
    const float c = p.scale_log2;
    // The k-th item of this CTA, as the loader published it: its index in the list, -1 when the list is exhausted,
    // -2 when the wait ran out.  Every consumer role reads every item and then gives the ring slot back.
    auto item_wait = [&](uint32_t k) -> int {
        if (!mbar_wait(smem_addr(&sh.item_full[k & 3u]), (k >> 2) & 1u, wctx, kSiteItem)) return -2;
        return *reinterpret_cast<volatile int*>(&sh.item_ring[k & 3u]);
    };
    auto item_release = [&](uint32_t k) { mbar_arrive(smem_addr(&sh.item_empty[k & 3u])); };

    if (warp < 8) {
        // ============================================================ softmax of K/V tiles j = g, g+2, ... of every item
        setmaxnreg_inc<kSpRegsSoftmax>();
        const int g = warp >> 2;
        const int row = tid & (kTileM - 1);
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + Cfg::kColS + g * 128 + lane_sel;
        const uint32_t tP = tmem_base + Cfg::kColP + g * 64 + lane_sel;
        const uint32_t bar_s = smem_addr(&sh.s_full[g]);
        const uint32_t bar_sf = smem_addr(&sh.s_free[g]);
        const uint32_t bar_st = smem_addr(&sh.st_full[g]);
        const uint32_t bar_st_other = smem_addr(&sh.st_full[g ^ 1]);
        const uint32_t bar_pr = smem_addr(&sh.p_ready[g]);
        const uint32_t bar_pf = smem_addr(&sh.p_free[g]);
        const float tau_raw = kRescaleThresholdLog2 / c;
        uint32_t T = 0;                       // K/V tiles of the items before the current one
        uint32_t itc = 0;                     // items with K/V tiles finished so far
        bool ok = true;

        for (uint32_t k = 0; ok; ++k) {
            int idx = item_wait(k);
            idx = __shfl_sync(0xffffffffu, idx, 0);
            __syncwarp();
            if (lane == 0 && idx != -2) item_release(k);
            if (idx < 0) { ok = (idx == -1); break; }
            int n_kv, kmax_row;
            {
                StreamItem it;
                decode(idx, it);
                n_kv = it.n_kv;
                kmax_row = Sk - 1;
                if (p.causal && it.i0 + row + off < kmax_row) kmax_row = it.i0 + row + off;
            }
            if (n_kv == 0) {              // no key visible to any row of this tile: no loads, no MMAs, no barriers
                StreamItem it;
                decode(idx, it);
                const int i_glob = it.i0 + row;
                const bool row_valid = i_glob < Sq;
                const size_t lse_row0 = static_cast<size_t>(it.b * p.Hq + it.hq) * p.Sq;
                const long long o_base = it.b * p.o_stride_b + it.hq * p.o_stride_h;
                if (g == 0 && row_valid) {
                    __nv_bfloat16* o_row = p.O + (o_base + static_cast<long long>(i_glob) * p.o_stride_s);
                    const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int v = 0; v < DV / 8; ++v) reinterpret_cast<uint4*>(o_row)[v] = z;
                    if (p.lse) p.lse[lse_row0 + i_glob] = -INFINITY;
                }
                continue;
            }

            // the epilogue of the item before has read the row state in shared memory before any warp publishes the
            // state of this item's tiles; normally long complete
            if (itc >= 1u) {
                ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.state_read), (itc - 1u) & 1u, wctx, kSiteEpiState));
                if (!ok) break;
            }
            float l = 0.f;             // this warpgroup's partial row sum, relative to the current u
            for (int j = static_cast<int>((static_cast<uint32_t>(g) ^ T) & 1u); j < n_kv; j += 2) {      // tiles with (T + j) & 1 == g
                const uint32_t use = (T + static_cast<uint32_t>(j)) >> 1;       // n-th use of this warpgroup's buffers
                ok = __all_sync(0xffffffffu, mbar_wait(bar_s, use & 1u, wctx, kSiteSoftmaxSFull));
                if (!ok) break;
                tc_fence_after_sync();
                const int j0 = j * kTileN;
                const bool need_mask = (j0 + kTileN - 1 > kmax_row);

                uint32_t s[kTileN];
                tmem_ld_x32(tS + 0, s + 0);
                tmem_ld_x32(tS + 32, s + 32);
                tmem_ld_x32(tS + 64, s + 64);
                tmem_ld_x32(tS + 96, s + 96);
                tc_wait_ld();
                // S^g is in registers: the score MMA of the buffer's next use may overwrite it
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_sf);
                if (need_mask) {
#pragma unroll
                    for (int e = 0; e < kTileN; ++e)
                        if (j0 + e > kmax_row) s[e] = 0xff800000u;   // -inf
                }
                float a[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) a[q] = -INFINITY;
#pragma unroll
                for (int e = 0; e < kTileN; e += 16) {
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        a[q] = fmax3(a[q], __uint_as_float(s[e + 2 * q]), __uint_as_float(s[e + 2 * q + 1]));
                }
                float mx = fmaxf(fmax3(a[0], a[1], a[2]), fmax3(a[3], a[4], a[5]));
                mx = fmax3(mx, a[6], a[7]);

                // Row state of tile j-1 (the other warpgroup's): u, and the factor r it applied.
                float m_ref = -INFINITY, r_prev = 1.f;
                if (j > 0) {
                    const uint32_t use_prev = (T + static_cast<uint32_t>(j - 1)) >> 1;
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_st_other, use_prev & 1u, wctx, kSiteSoftmaxCorrFree));
                    if (!ok) break;
                    m_ref = sh.mref[row];
                    r_prev = sh.alpha[g ^ 1][row];
                }
                // P^g and the slot of this tile's r are reused: the PV MMA of the buffer's previous use (two tiles
                // ago, or in the item before) must be complete, which also means that the correction warps have
                // consumed its r (see fa_fwd_stream.cuh).
                if (use >= 1u) {
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_pf, (use - 1u) & 1u, wctx, kSiteSoftmaxPFree));
                    if (!ok) break;
                }
                float alpha = 1.f;
                if (mx > m_ref + tau_raw) {
                    alpha = exp2_approx((m_ref - mx) * c);    // r = exp(u' - u); 0 on the first tile
                    m_ref = mx;
                }
                sh.mref[row] = m_ref;
                sh.alpha[g][row] = alpha;
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_st);

                const float mc = (m_ref == -INFINITY) ? 0.f : m_ref * c;
                const float2 c2 = make_float2(c, c);
                const float2 nmc2 = make_float2(-mc, -mc);
                float2 sum_a = make_float2(0.f, 0.f), sum_b = make_float2(0.f, 0.f);
                auto exp_chunk = [&](int q) {
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[q * 32 + e]),
                                                                __uint_as_float(s[q * 32 + e + 1])), c2, nmc2);
                        s[q * 32 + e] = __float_as_uint(exp2_approx(x.x));
                        s[q * 32 + e + 1] = __float_as_uint(exp2_approx(x.y));
                    }
                };
                auto emit_chunk = [&](int q) {
                    uint32_t pk[16];
#pragma unroll
                    for (int e = 0; e < 32; e += 4) {
                        const float2 v0 = make_float2(__uint_as_float(s[q * 32 + e]), __uint_as_float(s[q * 32 + e + 1]));
                        const float2 v1 = make_float2(__uint_as_float(s[q * 32 + e + 2]), __uint_as_float(s[q * 32 + e + 3]));
                        sum_a = __fadd2_rn(sum_a, v0);
                        sum_b = __fadd2_rn(sum_b, v1);
                        pk[e / 2] = pack_bf16x2(v0.x, v0.y);
                        pk[e / 2 + 1] = pack_bf16x2(v1.x, v1.y);
                    }
                    tmem_st_x16(tP + q * 16, pk);
                };
                exp_chunk(0);
                exp_chunk(1);
                emit_chunk(0);
                exp_chunk(2);
                emit_chunk(1);
                exp_chunk(3);
                emit_chunk(2);
                emit_chunk(3);
                l = l * (r_prev * alpha) + ((sum_a.x + sum_a.y) + (sum_b.x + sum_b.y));
                tc_wait_st();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_pr);
            }
            if (!ok) break;

            // ---- end of the item: the partial row sum goes to the correction warps, which run the epilogue
            const int last = n_kv - 1;
            // The warpgroup that did not run the last tile still has to apply its r.
            const int g_last = static_cast<int>((T + static_cast<uint32_t>(last)) & 1u);      // the warpgroup of the last tile
            if (g_last != g && last >= 1) {
                const uint32_t use_last = (T + static_cast<uint32_t>(last)) >> 1;
                ok = __all_sync(0xffffffffu, mbar_wait(bar_st_other, use_last & 1u, wctx, kSiteSoftmaxCorrFree));
                if (ok) l *= sh.alpha[g_last][row];
            }
            if (!ok) break;
            sh.lsum[g][row] = (last >= 1 || g_last == g) ? l : 0.f;       // (a single tile belongs to one warpgroup only)
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_addr(&sh.l_ready));
            T += static_cast<uint32_t>(n_kv);
            ++itc;
        }
    } else if (warp < 12) {
        // ============================================================ correction of the O accumulator
        setmaxnreg_dec<kSpRegsCorrection>();
        const int row = tid & (kTileM - 1);
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tO = tmem_base + Cfg::kColO + lane_sel;
        uint32_t T = 0;                       // K/V tiles of the items before the current one
        uint32_t vt = 0, itc = 0;             // V ring positions taken and items finished before the current item
        bool ok = true;
        for (uint32_t k = 0; ok; ++k) {
            int idx = item_wait(k);
            idx = __shfl_sync(0xffffffffu, idx, 0);
            __syncwarp();
            if (lane == 0 && idx != -2) item_release(k);
            if (idx < 0) break;
            StreamItem it;
            decode(idx, it);
            if (it.n_kv == 0) continue;
            const int n_kv = it.n_kv;
            for (int j = 0; j < n_kv && ok; ++j) {
                const uint32_t gj = T + static_cast<uint32_t>(j), bsel = gj & 1u, use = gj >> 1;
                ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.st_full[bsel]), use & 1u, wctx, kSiteCorrScale));
                if (!ok) break;
                const float alpha = sh.alpha[bsel][row];
                if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                    // O must hold the complete sum up to tile j-1 before it is rescaled
                    const uint32_t use_prev = (gj - 1u) >> 1;
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.p_free[bsel ^ 1u]), use_prev & 1u, wctx, kSiteCorrPvDone));
                    if (!ok) break;
                    tc_fence_after_sync();
#pragma unroll 1
                    for (int cc = 0; cc < DV / 32; ++cc) {
                        uint32_t r[32];
                        tmem_ld_x32(tO + cc * 32, r);
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                        tmem_st_x32(tO + cc * 32, r);
                    }
                    tc_wait_st();
                    tc_fence_before_sync();
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_addr(&sh.p_ready[bsel]));
            }
            if (!ok) break;

            // ---- epilogue of the item: O = G' / s (bf16), lse = u * scale + ln s
            const uint32_t ipar = itc & 1u;
            ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.l_ready), ipar, wctx, kSiteEpiStaged));
            if (!ok) break;
            const float lt = sh.lsum[0][row] + sh.lsum[1][row];
            const float m_fin = sh.mref[row];
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_addr(&sh.state_read));        // the softmax warps may publish the next item's state
            ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.o_final), ipar, wctx, kSiteEpiOFull));
            if (!ok) break;
            tc_fence_after_sync();
            const int i_glob = it.i0 + row;
            const float inv_l = (lt > 0.f) ? (1.f / lt) : 0.f;
            if (p.lse && i_glob < Sq)
                p.lse[static_cast<size_t>(it.b * p.Hq + it.hq) * p.Sq + i_glob] =
                    (lt > 0.f) ? (m_fin * c * 0.6931471805599453f + logf(lt)) : -INFINITY;
            // O goes into the staging tile (the V stage after the item's last V tile: its previous tile was read by a PV
            // product that is complete), then one thread stores it with TMA; rows past Sq are clipped
            const int s_stage = static_cast<int>((vt + static_cast<uint32_t>(n_kv)) % NV);
            const uint32_t s_tile = sV + s_stage * Cfg::kVBytes;
            const uint32_t sO = s_tile + row * 128;
#pragma unroll 1
            for (int cc = 0; cc < DV / 32; ++cc) {
                uint32_t r[32];
                tmem_ld_x32(tO + cc * 32, r);
                tc_wait_ld();
                const uint32_t chunk = sO + (cc >> 1) * kChunkBytes;
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const uint32_t piece = static_cast<uint32_t>(((cc & 1) * 4 + v) ^ (row & 7)) << 4;
                    st_shared_v4(chunk + piece,
                                 pack_bf16x2(__uint_as_float(r[8 * v]) * inv_l, __uint_as_float(r[8 * v + 1]) * inv_l),
                                 pack_bf16x2(__uint_as_float(r[8 * v + 2]) * inv_l, __uint_as_float(r[8 * v + 3]) * inv_l),
                                 pack_bf16x2(__uint_as_float(r[8 * v + 4]) * inv_l, __uint_as_float(r[8 * v + 5]) * inv_l),
                                 pack_bf16x2(__uint_as_float(r[8 * v + 6]) * inv_l, __uint_as_float(r[8 * v + 7]) * inv_l));
                }
            }
            // O is out of TMEM: the next item's first PV product may overwrite it
            tc_fence_before_sync();
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_addr(&sh.o_read));
                mbar_arrive(smem_addr(&sh.o_staged));
            }
            if (warp == 8 && lane == 0) {
                if (mbar_wait(smem_addr(&sh.o_staged), ipar, wctx, kSiteEpiStaged)) {
#pragma unroll
                    for (int ch = 0; ch < DV / kChunkCols; ++ch)
                        tma_store_4d(&tm_o, s_tile + ch * kChunkBytes, ch * kChunkCols, it.i0, it.hq, it.b);
                    tma_store_commit();
                    tma_store_wait_read_all();     // the staging tile goes back to the V ring
                    mbar_arrive(smem_addr(&sh.v_empty[s_stage]));
                }
            }
            __syncwarp();
            vt += static_cast<uint32_t>(n_kv) + 1u;
            ++itc;
            T += static_cast<uint32_t>(n_kv);
        }
    } else if (warp == 12) {
        // ============================================================ score MMAs: S^(j&1) = Q K_j^T
        setmaxnreg_dec<kSpRegsOther>();
        if (elect_one()) {
            constexpr uint32_t kIdescQK = make_idesc_bf16_f32(kTileM, kTileN, false, false);
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // sbo, version, swizzle
            const uint32_t q_lo = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
            auto desc = [](uint32_t lo) -> uint64_t { return (static_cast<uint64_t>(kDescHi) << 32) | lo; };
            uint32_t T = 0;
            uint32_t itc = 0;
            int sk = 0;
            uint32_t ph_k = 0;
            bool ok = true;
            for (uint32_t k = 0; ok; ++k) {
                const int idx = item_wait(k);
                if (idx != -2) item_release(k);
                if (idx < 0) break;
                StreamItem it;
                decode(idx, it);
                if (it.n_kv == 0) continue;
                const int n_kv = it.n_kv;
                ok = mbar_wait(smem_addr(&sh.q_full), itc & 1u, wctx, kSiteMmaQFull);
                for (int j = 0; j < n_kv && ok; ++j) {
                    const uint32_t gj = T + static_cast<uint32_t>(j), bsel = gj & 1u, use = gj >> 1;
                    ok = mbar_wait(smem_addr(&sh.k_full[sk]), ph_k, wctx, kSiteMmaKvFull);
                    // the softmax warps have read the buffer's previous S (two tiles ago, or in the item before)
                    if (ok && use >= 1u) ok = mbar_wait(smem_addr(&sh.s_free[bsel]), (use - 1u) & 1u, wctx, kSiteMmaSFree);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t tS = tmem_base + Cfg::kColS + bsel * 128;
                    const uint32_t klo = k_lo0 + sk * (Cfg::kKBytes >> 4);
#pragma unroll
                    for (int k = 0; k < DQK / 16; ++k) {
                        const uint32_t koff = ((k / 4) * kChunkBytes + (k % 4) * 32) >> 4;
                        mma_ss(tS, desc(q_lo + koff), desc(klo + koff), kIdescQK, k > 0 ? 1u : 0u);
                    }
                    tc_commit(smem_addr(&sh.s_full[bsel]));
                    tc_commit(smem_addr(&sh.k_empty[sk]));
                    if (j + 1 == n_kv) tc_commit(smem_addr(&sh.q_free));
                    if (++sk == NK) { sk = 0; ph_k ^= 1u; }
                }
                T += static_cast<uint32_t>(n_kv);
                ++itc;
            }
        }
    } else if (warp == 13) {
        // ============================================================ PV MMAs: O += P^(j&1) V_j
        setmaxnreg_dec<kSpRegsOther>();
        if (elect_one()) {
            constexpr uint32_t kIdescPV = make_idesc_bf16_f32(kTileM, DV, false, true);
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
            const uint32_t v_lo0 = ((sV & 0x3FFFFu) >> 4) | ((static_cast<uint32_t>(kChunkBytes) >> 4) << 16);
            const uint32_t tO = tmem_base + Cfg::kColO;
            auto desc = [](uint32_t lo) -> uint64_t { return (static_cast<uint64_t>(kDescHi) << 32) | lo; };
            uint32_t T = 0;
            uint32_t itc = 0;
            int sv = 0;
            uint32_t ph_v = 0;
            bool ok = true;
            for (uint32_t k = 0; ok; ++k) {
                const int idx = item_wait(k);
                if (idx != -2) item_release(k);
                if (idx < 0) break;
                StreamItem it;
                decode(idx, it);
                if (it.n_kv == 0) continue;
                const int n_kv = it.n_kv;
                // the epilogue of the item before has read O out of TMEM
                if (itc >= 1u) ok = mbar_wait(smem_addr(&sh.o_read), (itc - 1u) & 1u, wctx, kSiteMmaSFree);
                for (int j = 0; j < n_kv && ok; ++j) {
                    const uint32_t gj = T + static_cast<uint32_t>(j), bsel = gj & 1u, use = gj >> 1;
                    ok = mbar_wait(smem_addr(&sh.v_full[sv]), ph_v, wctx, kSiteMmaKvFull);
                    if (ok) ok = mbar_wait(smem_addr(&sh.p_ready[bsel]), use & 1u, wctx, kSiteMmaPFull);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t tP = tmem_base + Cfg::kColP + bsel * 64;
                    const uint32_t vlo = v_lo0 + sv * (Cfg::kVBytes >> 4);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        mma_ts(tO, tP + kk * 8, desc(vlo + kk * (2048 >> 4)), kIdescPV, (j > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(smem_addr(&sh.p_free[bsel]));
                    tc_commit(smem_addr(&sh.v_empty[sv]));
                    if (j + 1 == n_kv) tc_commit(smem_addr(&sh.o_final));
                    if (++sv == NV) { sv = 0; ph_v ^= 1u; }
                }
                if (++sv == NV) { sv = 0; ph_v ^= 1u; }       // the ring position of the item's staging tile
                T += static_cast<uint32_t>(n_kv);
                ++itc;
            }
        }
    } else if (warp == 14) {
        // ============================================================ TMA loads of Q and K
        setmaxnreg_dec<kSpRegsOther>();
        if (elect_one()) {
            uint32_t itc = 0;
            uint32_t kt = 0;                  // K tiles loaded so far (ring position)
            bool ok = true;
            auto load_k = [&](const StreamItem& it, int j) -> bool {
                const int s = static_cast<int>(kt % NK);
                if (!mbar_wait(smem_addr(&sh.k_empty[s]), ((kt / NK) & 1u) ^ 1u, wctx, kSiteLoadKvEmpty)) return false;
                const uint32_t bar = smem_addr(&sh.k_full[s]);
                mbar_arrive_expect_tx(bar, Cfg::kKBytes);
#pragma unroll
                for (int cc = 0; cc < Cfg::kQChunks; ++cc)
                    tma_load_4d(sK + s * Cfg::kKBytes + cc * kChunkBytes, &tm_k, bar, cc * kChunkCols, j * kTileN, it.kvh, it.b);
                ++kt;
                return true;
            };
            int idx = cta;                    // the first item; every further one by ticket
            for (uint32_t k = 0; ok; ++k) {
                // publish the item (or the end of the list) to the other roles
                ok = mbar_wait(smem_addr(&sh.item_empty[k & 3u]), ((k >> 2) & 1u) ^ 1u, wctx, kSiteItem);
                if (!ok) break;
                *reinterpret_cast<volatile int*>(&sh.item_ring[k & 3u]) = (idx < n_items) ? idx : -1;
                mbar_arrive(smem_addr(&sh.item_full[k & 3u]));      // (release: the store above is visible to whoever sees the phase)
                if (idx >= n_items) break;
                StreamItem it;
                decode(idx, it);
                // the next item is drawn now, one item ahead of the loads below; the launch makes n_items draws in all
                // (every CTA draws until the list is exhausted), and the CTA that makes the last one zeroes the counter
                {
                    const unsigned int ticket = atomicAdd(p.sched_counter, 1u);
                    if (ticket == static_cast<unsigned int>(n_items) - 1u) atomicExch(p.sched_counter, 0u);
                    idx = G + static_cast<int>(ticket);
                }
                if (it.n_kv == 0) continue;
                const int n_kv = it.n_kv;
                // the first K tiles go ahead of Q: their stages are free before the query tile's space is (the last one
                // of the ring comes free with it: both were read by the last score MMA of the item before)
                const int ahead = n_kv < NK - 1 ? n_kv : NK - 1;
                for (int j = 0; j < ahead && ok; ++j) ok = load_k(it, j);
                if (!ok) break;
                // the last score MMA of the item before has read the query tile
                if (itc >= 1u) ok = mbar_wait(smem_addr(&sh.q_free), (itc - 1u) & 1u, wctx, kSiteLoadKvEmpty);
                if (!ok) break;
                {
                    const uint32_t bar = smem_addr(&sh.q_full);
                    mbar_arrive_expect_tx(bar, static_cast<uint32_t>(Cfg::kQBytes));
#pragma unroll
                    for (int cc = 0; cc < Cfg::kQChunks; ++cc)
                        tma_load_4d(sQ + cc * kChunkBytes, &tm_q, bar, cc * kChunkCols, it.i0, it.hq, it.b);
                }
                for (int j = ahead; j < n_kv && ok; ++j) ok = load_k(it, j);
                ++itc;
            }
        }
    } else {
        // ============================================================ warp 15: TMA loads of V
        setmaxnreg_dec<kSpRegsOther>();
        if (elect_one()) {
            uint32_t vt = 0;                  // V tiles that have gone through the ring
            bool first = true;
            bool ok = true;
            for (uint32_t k = 0; ok; ++k) {
                const int idx = item_wait(k);
                if (idx != -2) item_release(k);
                if (idx < 0) break;
                StreamItem it;
                decode(idx, it);
                if (it.n_kv == 0) continue;
                for (int j = 0; j < it.n_kv && ok; ++j) {
                    if (p.debug_drop_v_load && first) { first = false; ok = false; break; }      // (test hook: see FA_FLAG_DEBUG_DROP_V_LOAD)
                    const int s = static_cast<int>(vt % NV);
                    ok = mbar_wait(smem_addr(&sh.v_empty[s]), ((vt / NV) & 1u) ^ 1u, wctx, kSiteLoadKvEmpty);
                    if (!ok) break;
                    const uint32_t bar = smem_addr(&sh.v_full[s]);
                    mbar_arrive_expect_tx(bar, Cfg::kVBytes);
#pragma unroll
                    for (int cc = 0; cc < Cfg::kVChunks; ++cc)
                        tma_load_4d(sV + s * Cfg::kVBytes + cc * kChunkBytes, &tm_v, bar, cc * kChunkCols, j * kTileN, it.kvh, it.b);
                    ++vt;
                }
                if (!ok) break;
                {
                    // The ring position of the item's staging tile: nothing to load, but the stage's barriers move on
                    // in step with the positions (a plain arrival completes the phase of v_full that a load would
                    // have; it may only be made once the stage's previous phase is over, i.e. its tile consumed).
                    const int s = static_cast<int>(vt % NV);
                    ok = mbar_wait(smem_addr(&sh.v_empty[s]), ((vt / NV) & 1u) ^ 1u, wctx, kSiteLoadKvEmpty);
                    if (!ok) break;
                    mbar_arrive(smem_addr(&sh.v_full[s]));
                    ++vt;
                }
            }
        }
    }

    // ---------------------------------------------------------------- teardown (all warps)
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 12) tmem_dealloc(tmem_base, Cfg::kTmemCols);
}

}  // namespace fa
