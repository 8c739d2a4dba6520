// Persistent form of the head-size-128 pair kernel for sm_100a: one CTA per SM walks a list of work items
// (item = two query tiles, as in fa_fwd_pair.cuh), with the inner loop of fa_fwd_pair.cuh and the item
// machinery of fa_fwd_persistent.cuh.  Read those two files first; this one only joins them.
//
// From fa_fwd_pair.cuh: one elected thread issues the MMAs of both tiles in a fixed order, the barriers
// it needs next are probed from inside the blocks of MMAs, there is no correction warpgroup (the softmax
// warps rescale their own rows of O_t on the rare tiles where the reference maximum moves), P_t is
// handed over as keys 0..95 and 96..127, the row sum is taken after the hand-off.
// From fa_fwd_persistent.cuh: items are ordered longest first, CTA c starts with item c and draws every
// further item from a global ticket counter (the K/V load thread, once the loads of its current item
// are issued); that thread decodes the item once and passes it to the other roles through a four-slot
// ring; Q tiles have a loader of their own that refills Q_t as soon as the item's last score MMA of
// that tile is complete; O leaves through a staging buffer (two K stages instead of three pay for it),
// so that between the last P_t V of one item and the first softmax of the next a tile only has the
// read-out of O_t.  All mbarrier phases and ring stages run on across items; inside an item the MMA
// thread's probes work as in the pair kernel, at an item's start it waits the ordinary way.
//
// Results are bit-identical to fa_fwd_pair_kernel and fa_fwd_persistent_kernel (same MMAs in the same
// order per accumulator, same softmax arithmetic).
//
// Roles (384 threads): warps 0-3 / 4-7 softmax and epilogue of tile 0 / 1, warp 8 MMA issue, warp 9 K/V
// loads, item draw and decode, warp 10 Q loads, warp 11 idle.
#pragma once

#include "fa_fwd_pair.cuh"
#include "fa_fwd_persistent.cuh"

namespace fa {

struct PairPersistCfg {
    static constexpr int kQBytes = 2 * kChunkBytes;       // one 128 x 128 bf16 tile
    static constexpr int kKBytes = kQBytes, kVBytes = kQBytes, kOBytes = kQBytes;
    static constexpr int kKStages = 2, kVStages = 2;
    static constexpr int kTileBytes = 2 * kQBytes + kKStages * kKBytes + kVStages * kVBytes + kOBytes;
    static constexpr int kTmemCols = 512;
    static constexpr int kColS0 = 0, kColS1 = 128, kColO0 = 256, kColO1 = 384;
    static constexpr int kThreads = 384;
};

struct PairPersistShared {
    uint64_t q_full[2], q_empty[2];
    uint64_t k_full[4], k_empty[4];
    uint64_t v_full[4], v_empty[4];
    uint64_t s_full[2];      // MMA -> softmax: S_t(j) is in TMEM
    uint64_t p_first[2];     // softmax -> MMA: keys 0..95 of P_t(j) written, O_t rescaled if it had to be
    uint64_t p_rest[2];      // softmax -> MMA: all of P_t(j) written
    uint64_t o_final[2];     // MMA -> softmax: last PV of tile t of the item done
    uint64_t stage_full;     // softmax warps -> storing thread: the bf16 O tile is in the staging buffer
    uint64_t stage_empty;    // storing thread -> softmax warps: the TMA store has read the staging buffer
    uint64_t item_full[4];   // K/V load thread -> every role: items[slot] holds the next work item
    uint64_t item_empty[4];  // every role -> K/V load thread: slot read (8 softmax warps, MMA thread, Q loader)
    int item_ring[4];        // index of the item in the list (>= the list's length: the end mark)
    PersistItem items[4];
    uint32_t tmem_base;
    uint32_t abort_flag;
};

constexpr int pair_persist_smem_bytes() {
    return PairPersistCfg::kTileBytes + static_cast<int>(sizeof(PairPersistShared));
}

template <bool kVarlen = false>
__global__ void __launch_bounds__(384, 1)
fa_fwd_pair_persistent_kernel(const __grid_constant__ CUtensorMap tm_q,
                              const __grid_constant__ CUtensorMap tm_k,
                              const __grid_constant__ CUtensorMap tm_v,
                              const __grid_constant__ CUtensorMap tm_o,
                              const FwdParams p) {
    using Cfg = PairPersistCfg;
    using namespace ptx;
    constexpr int DQK = 128, DV = 128;
    constexpr int NK = Cfg::kKStages;
    constexpr int NV = Cfg::kVStages;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    PairPersistShared& sh = *reinterpret_cast<PairPersistShared*>(smem_raw + Cfg::kTileBytes);

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
    const uint32_t sQ = smem_base;                               // two tiles
    const uint32_t sK = sQ + 2 * Cfg::kQBytes;                   // NK stages
    const uint32_t sV = sK + NK * Cfg::kKBytes;                  // NV stages
    const uint32_t sStage = sV + NV * Cfg::kVBytes;              // one bf16 output tile

    const int n_items = p.head_pair ? p.n_q_tiles * p.B * (p.Hq / 2) : ((p.n_q_tiles + 1) / 2) * p.B * p.Hq;
    const int G = static_cast<int>(gridDim.x);
    const int cta = static_cast<int>(blockIdx.x);

    // ---------------------------------------------------------------- setup
    if (tid == 0) {
        sh.abort_flag = 0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_addr(&sh.q_full[t]), 1);
            mbar_init(smem_addr(&sh.q_empty[t]), 1);
            mbar_init(smem_addr(&sh.s_full[t]), 1);
            mbar_init(smem_addr(&sh.p_first[t]), 4);      // 4 softmax warps
            mbar_init(smem_addr(&sh.p_rest[t]), 4);
            mbar_init(smem_addr(&sh.o_final[t]), 1);
        }
        mbar_init(smem_addr(&sh.stage_full), 4);          // 4 softmax warps of the tile being stored
        mbar_init(smem_addr(&sh.stage_empty), 1);
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            mbar_init(smem_addr(&sh.item_full[s]), 1);
            mbar_init(smem_addr(&sh.item_empty[s]), 10);
            mbar_init(smem_addr(&sh.k_full[s]), 1);
            mbar_init(smem_addr(&sh.k_empty[s]), 1);
            mbar_init(smem_addr(&sh.v_full[s]), 1);
            mbar_init(smem_addr(&sh.v_empty[s]), 1);
        }
        fence_mbar_init();
    }
    if (warp == 8) {
        tmem_alloc(smem_addr(&sh.tmem_base), Cfg::kTmemCols);
        tmem_relinquish_alloc_permit();
    }
    if (warp == 9 && lane == 0) {
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

    // Consumer side of the work-item ring, as in fa_fwd_persistent_kernel.
    auto item_wait_thread = [&](int k) -> int {
        const int slot = k & 3;
        if (!mbar_wait(smem_addr(&sh.item_full[slot]), (static_cast<uint32_t>(k) >> 2) & 1u, wctx, kSiteItem)) return -1;
        const int idx = *reinterpret_cast<volatile int*>(&sh.item_ring[slot]);
        return idx < n_items ? idx : -1;
    };
    auto item_wait = [&](int k) -> int {
        const int slot = k & 3;
        if (!__all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.item_full[slot]), (static_cast<uint32_t>(k) >> 2) & 1u,
                                               wctx, kSiteItem))) return -1;
        const int idx = *reinterpret_cast<volatile int*>(&sh.item_ring[slot]);
        return idx < n_items ? idx : -1;
    };
    auto item_at = [&](int k) -> PersistItem {
        PersistItem it_;
        const volatile int4* src = reinterpret_cast<const volatile int4*>(&sh.items[k & 3]);
        int4* dst = reinterpret_cast<int4*>(&it_);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            dst[i].x = src[i].x; dst[i].y = src[i].y; dst[i].z = src[i].z; dst[i].w = src[i].w;
        }
        return it_;
    };
    auto item_release_thread = [&](int k) { mbar_arrive(smem_addr(&sh.item_empty[k & 3])); };
    auto item_release = [&](int k) {
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_addr(&sh.item_empty[k & 3]));
    };

    if (warp < 8) {
        // ============================================================ softmax of tile t
        setmaxnreg_inc<kPairRegsSoftmax>();
        const int t = warp >> 2;
        const int row = tid & (kTileM - 1);
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + (t == 0 ? Cfg::kColS0 : Cfg::kColS1) + lane_sel;
        const uint32_t tO = tmem_base + (t == 0 ? Cfg::kColO0 : Cfg::kColO1) + lane_sel;
        const uint32_t bar_s = smem_addr(&sh.s_full[t]);
        const uint32_t bar_pf = smem_addr(&sh.p_first[t]);
        const uint32_t bar_pr = smem_addr(&sh.p_rest[t]);
        const float tau_raw = kRescaleThresholdLog2 / c;
        uint32_t it = 0;       // iterations of this tile so far, over all items: barrier parities
        uint32_t oc = 0;       // items with work for this tile so far: parity of o_final
        uint32_t uc = 0;       // uses of the staging buffer so far, by either tile
        bool ok = true;
        FA_PHASE_DECL();       // phases: 0 wait for the item, 1 wait for S, 2 softmax pass, 3 wait for the last PV, 4 wait for the staging buffer, 5 read-out of O, 6 store
        int n_done = 0;

#pragma unroll 1
        for (int k = 0; ok; item_release(k), ++k) {      // (the slot is kept until the item's epilogue has read it again)
            if (item_wait(k) < 0) break;
            FA_PHASE(0);
            ++n_done;
            int nkv_t, i0_t, Sq, Sk;
            uint32_t my_use;           // this tile's place in the order of staging-buffer users
            {
                const PersistItem item = item_at(k);
                nkv_t = t == 0 ? item.nkv_0 : item.nkv_1;
                i0_t = t == 0 ? item.i0_0 : item.i0_1;
                Sq = item.Sq;
                Sk = item.Sk;
                my_use = uc + ((t == 1 && item.nkv_0 > 0) ? 1u : 0u);
                uc += (item.nkv_0 > 0 ? 1u : 0u) + (item.nkv_1 > 0 ? 1u : 0u);
            }
            const int i_glob = i0_t + row;
            const int off = Sk - Sq;
            int kmax_row = Sk - 1;
            if (p.causal && i_glob + off < kmax_row) kmax_row = i_glob + off;

            float m_ref = -INFINITY;   // reference maximum, raw score units
            float l = 0.f;
#pragma unroll 1
            for (int j = 0; j < nkv_t; ++j, ++it) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar_s, it & 1u, wctx, kSiteSoftmaxSFull));
                if (!ok) break;
                FA_PHASE(1);
                tc_fence_after_sync();
                softmax_pass_128<DV>(tS, tO, c, tau_raw, j * kTileN, kmax_row, j == 0, m_ref, l, lane,
                                     [&]() { mbar_arrive(bar_pf); }, [&]() { mbar_arrive(bar_pr); });
                FA_PHASE(2);
            }
            if (!ok) break;

            // ---- epilogue of the item: O = G' / s (bf16), lse = u * scale + ln s   (as in fa_fwd_persistent_kernel)
            if (i0_t >= Sq) continue;
            const PersistItem item = item_at(k);     // again: nothing of it was kept live
            const int hq_t = t == 0 ? item.hq : item.hq1;
            const size_t lse_row0 = kVarlen ? static_cast<size_t>(hq_t) * p.total_q + item.q_row0
                                            : (static_cast<size_t>(item.b) * p.Hq + hq_t) * p.Sq;
            __nv_bfloat16* o_row = p.O + ((kVarlen ? item.q_row0 * p.o_stride_s : item.b * p.o_stride_b) + hq_t * p.o_stride_h +
                                          static_cast<long long>(i_glob) * p.o_stride_s);
            if (nkv_t == 0) {             // no key visible to any row of this tile
                if (i_glob < Sq) {
                    const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int v = 0; v < DV / 8; ++v) reinterpret_cast<uint4*>(o_row)[v] = z;
                    if (p.lse) p.lse[lse_row0 + i_glob] = -INFINITY;
                }
                continue;
            }
            ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.o_final[t]), oc & 1u, wctx, kSiteEpiOFull));
            ++oc;
            if (!ok) break;
            FA_PHASE(3);
            tc_fence_after_sync();
            const float inv_l = (l > 0.f) ? (1.f / l) : 0.f;
            if (p.lse && i_glob < Sq)
                p.lse[lse_row0 + i_glob] = (l > 0.f) ? (m_ref * c * 0.6931471805599453f + logf(l)) : -INFINITY;
            const bool box_store = !kVarlen || (i0_t + kTileM <= Sq);
            // the previous user's TMA store must have read the staging buffer
            ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.stage_empty), (my_use & 1u) ^ 1u, wctx, kSiteEpiStaged));
            if (!ok) break;
            FA_PHASE(4);
            const uint32_t sO = sStage + row * 128;
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
            if (!box_store) {
                // every warp copies the 32 rows it staged itself, whole rows per instruction
                __syncwarp();
                store_staged_rows<DV>(sStage, (warp & 3) * 32, Sq - i0_t, o_row - static_cast<long long>(row) * p.o_stride_s,
                                      p.o_stride_s, lane);
            }
            // O_t has been read: order the TMEM loads before the next item's MMAs into O_t and S_t
            tc_fence_before_sync();
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_addr(&sh.stage_full));
            FA_PHASE(5);
            if ((warp & 3) == 0 && lane == 0) {
                ok = mbar_wait(smem_addr(&sh.stage_full), my_use & 1u, wctx, kSiteEpiStaged);
                if (ok) {
                    if (box_store) {
#pragma unroll
                        for (int ch = 0; ch < DV / kChunkCols; ++ch)
                            tma_store_4d(&tm_o, sStage + ch * kChunkBytes, ch * kChunkCols, item.q_row0 + i0_t, hq_t,
                                         kVarlen ? 0 : item.b);
                        tma_store_commit();
                        tma_store_wait_read_all();
                    }
                    mbar_arrive(smem_addr(&sh.stage_empty));
                }
            }
            ok = __all_sync(0xffffffffu, ok);
            FA_PHASE(6);
        }
        FA_PHASE_STORE(7, n_done);
    } else if (warp == 8) {
        // ============================================================ MMA issue, one thread for both tiles
        setmaxnreg_dec<kPairRegsOther>();
        if (elect_one()) {
            constexpr uint32_t kIdescQK = make_idesc_bf16_f32(kTileM, kTileN, false, false);
            constexpr uint32_t kIdescPV = make_idesc_bf16_f32(kTileM, DV, false, true);
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // sbo, version, swizzle
            const uint32_t q_lo0 = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t v_lo0 = ((sV & 0x3FFFFu) >> 4) | ((static_cast<uint32_t>(kChunkBytes) >> 4) << 16);
            auto desc = [](uint32_t lo) -> uint64_t {
                return (static_cast<uint64_t>(kDescHi) << 32) | lo;
            };
            auto koff = [](int kk) -> uint32_t { return static_cast<uint32_t>(((kk / 4) * kChunkBytes + (kk % 4) * 32) >> 4); };
            // a barrier whose phase 0 completed at the first item and that is probed with the parity of a phase that
            // is always complete: filler for unused probe slots (item_full[0] moves only when slot 0 is refilled, and
            // a probe of parity p succeeds whenever the barrier's current phase has parity 1 - p; see below)
            int sk = 0, sv = 0;                  // stage of the next K tile and the next V tile to consume
            uint32_t ph_k = 0, ph_v = 0;
            uint32_t it0 = 0, it1 = 0;           // iterations with work for tile 0 / 1 so far: parities of s_full, p_first, p_rest
            uint32_t qc0 = 0, qc1 = 0;           // items with work for tile 0 / 1 so far: parity of q_full
            bool ok = true;
#pragma unroll 1
            for (int k = 0; ok; ++k) {
                if (item_wait_thread(k) < 0) break;
                int nkv_0, nkv_1, n_max;
                {
                    const PersistItem item = item_at(k);
                    nkv_0 = item.nkv_0; nkv_1 = item.nkv_1; n_max = item.n_max;
                }
                item_release_thread(k);
                if (n_max == 0) continue;
                // First score blocks of the item.  S_t is free (the tile's last softmax pass has read it and its
                // last PV was issued before this), O_t is not touched before the tile's first P arrives, which its
                // softmax warps only send after their epilogue has read O_t out.
                ok = mbar_wait(smem_addr(&sh.k_full[sk]), ph_k, wctx, kSiteMmaKvFull);
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int nkv_t = t == 0 ? nkv_0 : nkv_1;
                    if (ok && nkv_t > 0) {
                        ok = mbar_wait(smem_addr(&sh.q_full[t]), (t == 0 ? qc0 : qc1) & 1u, wctx, kSiteMmaQFull);
                        if (t == 0) ++qc0; else ++qc1;
                        if (ok) {
                            tc_fence_after_sync();
                            const uint32_t tS = tmem_base + (t == 0 ? Cfg::kColS0 : Cfg::kColS1);
                            const uint32_t q_lo = q_lo0 + t * (Cfg::kQBytes >> 4);
                            const uint32_t klo = k_lo0 + sk * (Cfg::kKBytes >> 4);
#pragma unroll
                            for (int kk = 0; kk < DQK / 16; ++kk)
                                mma_ss(tS, desc(q_lo + koff(kk)), desc(klo + koff(kk)), kIdescQK, kk > 0 ? 1u : 0u);
                            tc_commit(smem_addr(&sh.s_full[t]));
                            if (nkv_t == 1) tc_commit(smem_addr(&sh.q_empty[t]));     // that was the item's last score MMA of the tile
                        }
                    }
                }
                if (!ok) break;
                tc_commit(smem_addr(&sh.k_empty[sk]));
                if (++sk == NK) { sk = 0; ph_k ^= 1u; }
                // results of the probes made from inside the block before: P_0 / P_1 first part, V_j, K_{j+1}
                uint32_t pre_p0 = 0u, pre_p1 = 0u, pre_v = 0u, pre_k = 0u;

                // One tile's block of iteration j: PV_t(j), then QK_t(j+1).  (b0, par0) ... (b2, par2): barriers to
                // probe from inside the block (use0..2: whether the slot is used); the result lands in `probed`.
                auto tile_block = [&](auto tc, int j, int nkv_t, uint32_t itt, uint32_t pre_first, bool use0, uint32_t b0,
                                      uint32_t par0, bool use1, uint32_t b1, uint32_t par1, bool use2, uint32_t b2, uint32_t par2,
                                      uint32_t& probed) -> bool {
                    constexpr int t = decltype(tc)::value;
                    probed = 0u;
                    if (j >= nkv_t) return true;
                    const uint32_t tS = tmem_base + (t == 0 ? Cfg::kColS0 : Cfg::kColS1);   // P_t overlays it
                    const uint32_t tO = tmem_base + (t == 0 ? Cfg::kColO0 : Cfg::kColO1);
                    const uint32_t q_lo = q_lo0 + t * (Cfg::kQBytes >> 4);
                    const uint32_t vlo = v_lo0 + sv * (Cfg::kVBytes >> 4);
                    const uint32_t klo = k_lo0 + sk * (Cfg::kKBytes >> 4);
                    if (!pre_first && !mbar_wait(smem_addr(&sh.p_first[t]), itt & 1u, wctx, kSiteMmaPFull)) return false;
                    tc_fence_after_sync();
                    // PV k-steps 0..3, then the probe of p_rest under k-steps 4 and 5
                    mma_ts(tO, tS + 0, desc(vlo + 0 * (2048 >> 4)), kIdescPV, j > 0 ? 1u : 0u);
                    mma_ts(tO, tS + 8, desc(vlo + 1 * (2048 >> 4)), kIdescPV, 1u);
                    mma_ts(tO, tS + 16, desc(vlo + 2 * (2048 >> 4)), kIdescPV, 1u);
                    mma_ts(tO, tS + 24, desc(vlo + 3 * (2048 >> 4)), kIdescPV, 1u);
                    const uint32_t rest = probe_mma_ts2(smem_addr(&sh.p_rest[t]), itt & 1u, tO, tS + 32, desc(vlo + 4 * (2048 >> 4)),
                                                        tS + 40, desc(vlo + 5 * (2048 >> 4)), kIdescPV);
                    if (!rest && !mbar_wait(smem_addr(&sh.p_rest[t]), itt & 1u, wctx, kSiteMmaPFull)) return false;
                    tc_fence_after_sync();
                    mma_ts(tO, tS + 48, desc(vlo + 6 * (2048 >> 4)), kIdescPV, 1u);
                    mma_ts(tO, tS + 56, desc(vlo + 7 * (2048 >> 4)), kIdescPV, 1u);
                    if (j + 1 < nkv_t) {
                        mma_ss(tS, desc(q_lo + koff(0)), desc(klo + koff(0)), kIdescQK, 0u);
                        mma_ss(tS, desc(q_lo + koff(1)), desc(klo + koff(1)), kIdescQK, 1u);
                        mma_ss(tS, desc(q_lo + koff(2)), desc(klo + koff(2)), kIdescQK, 1u);
                        mma_ss(tS, desc(q_lo + koff(3)), desc(klo + koff(3)), kIdescQK, 1u);
                        // an unused slot probes this tile's own p_rest again, whose phase was just seen complete
                        const uint32_t self = smem_addr(&sh.p_rest[t]), self_par = itt & 1u;
                        probed = probe3_mma_ss3(use0 ? b0 : self, use0 ? par0 : self_par, use1 ? b1 : self, use1 ? par1 : self_par,
                                                use2 ? b2 : self, use2 ? par2 : self_par, tS, desc(q_lo + koff(4)),
                                                desc(klo + koff(4)), desc(q_lo + koff(5)), desc(klo + koff(5)), desc(q_lo + koff(6)),
                                                desc(klo + koff(6)), kIdescQK);
                        probed &= (use0 ? 1u : 0u) | (use1 ? 2u : 0u) | (use2 ? 4u : 0u);
                        mma_ss(tS, desc(q_lo + koff(7)), desc(klo + koff(7)), kIdescQK, 1u);
                        tc_commit(smem_addr(&sh.s_full[t]));
                        if (j + 2 == nkv_t) tc_commit(smem_addr(&sh.q_empty[t]));     // last score MMA of the item: Q_t may be replaced
                    } else {
                        tc_commit(smem_addr(&sh.o_final[t]));
                    }
                    return true;
                };

#pragma unroll 1
                for (int j = 0; j < n_max && ok; ++j) {
                    if (!pre_v) ok = mbar_wait(smem_addr(&sh.v_full[sv]), ph_v, wctx, kSiteMmaKvFull);
                    if (ok && j + 1 < n_max && !pre_k) ok = mbar_wait(smem_addr(&sh.k_full[sk]), ph_k, wctx, kSiteMmaKvFull);
                    if (!ok) break;
                    uint32_t probed;
                    // block of tile 0; probe: first part of P_1(j)
                    ok = tile_block(IntC<0>{}, j, nkv_0, it0, pre_p0, j < nkv_1, smem_addr(&sh.p_first[1]), it1 & 1u,
                                    false, 0u, 0u, false, 0u, 0u, probed);
                    if (!ok) break;
                    if (j < nkv_0) ++it0;
                    pre_p1 = probed & 1u;
                    // stage and phase of V_{j+1} and K_{j+2}
                    int sv_n = sv + 1; uint32_t ph_v_n = ph_v; if (sv_n == NV) { sv_n = 0; ph_v_n ^= 1u; }
                    int sk_n = sk + 1; uint32_t ph_k_n = ph_k; if (sk_n == NK) { sk_n = 0; ph_k_n ^= 1u; }
                    // block of tile 1; probes: first part of P_0(j+1), V_{j+1}, K_{j+2}
                    ok = tile_block(IntC<1>{}, j, nkv_1, it1, pre_p1, j + 1 < nkv_0, smem_addr(&sh.p_first[0]), it0 & 1u,
                                    j + 1 < n_max, smem_addr(&sh.v_full[sv_n]), ph_v_n,
                                    j + 2 < n_max, smem_addr(&sh.k_full[sk_n]), ph_k_n, probed);
                    if (!ok) break;
                    if (j < nkv_1) ++it1;
                    pre_p0 = probed & 1u;
                    pre_v = (probed >> 1) & 1u;
                    pre_k = (probed >> 2) & 1u;
                    tc_commit(smem_addr(&sh.v_empty[sv]));
                    if (j + 1 < n_max) tc_commit(smem_addr(&sh.k_empty[sk]));
                    sv = sv_n; ph_v = ph_v_n;
                    if (j + 1 < n_max) { sk = sk_n; ph_k = ph_k_n; }
                }
            }
        }
    } else if (warp == 9) {
        // ============================================================ TMA loads of K and V, item draw and decode
        setmaxnreg_dec<kPairRegsOther>();
        if (elect_one()) {
            uint32_t kc = 0, vc = 0;         // K and V tiles requested so far, over all items
            int idx = cta;                   // first item: static, the heaviest items go first
            bool ok = true;
#pragma unroll 1
            for (int k = 0; ok; ++k) {
                // publish the item (or the end mark) to the other roles
                const int slot = k & 3;
                if (k >= 4) ok = mbar_wait(smem_addr(&sh.item_empty[slot]), ((static_cast<uint32_t>(k) >> 2) - 1u) & 1u, wctx, kSiteItem);
                if (!ok) break;
                PersistItem item;
                if (idx < n_items) {
                    item = persist_decode<kVarlen>(p, idx);
                    item.pad[0] = item.pad[1] = item.pad[2] = 0;
                    const int4* src = reinterpret_cast<const int4*>(&item);
                    volatile int4* dst = reinterpret_cast<volatile int4*>(&sh.items[slot]);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        dst[i].x = src[i].x; dst[i].y = src[i].y; dst[i].z = src[i].z; dst[i].w = src[i].w;
                    }
                }
                *reinterpret_cast<volatile int*>(&sh.item_ring[slot]) = idx;
                mbar_arrive(smem_addr(&sh.item_full[slot]));       // (release: the stores above are visible to whoever sees the phase)
                if (idx >= n_items) break;
#pragma unroll 1
                for (int j = 0; j < item.n_max; ++j) {
                    const int j0 = j * kTileN;
                    {
                        const uint32_t s = kc % NK;
                        ok = mbar_wait(smem_addr(&sh.k_empty[s]), ((kc / NK) & 1u) ^ 1u, wctx, kSiteLoadKvEmpty);
                        if (!ok) break;
                        const uint32_t bar = smem_addr(&sh.k_full[s]);
                        mbar_arrive_expect_tx(bar, Cfg::kKBytes);
#pragma unroll
                        for (int cc = 0; cc < 2; ++cc)
                            tma_load_4d(sK + s * Cfg::kKBytes + cc * kChunkBytes, &tm_k, bar, cc * kChunkCols,
                                        item.k_row0 + j0, item.kvh, kVarlen ? 0 : item.b);
                        ++kc;
                    }
                    if (!(p.debug_drop_v_load && k == 0 && j == 0)) {      // (test hook: see FA_FLAG_DEBUG_DROP_V_LOAD)
                        const uint32_t s = vc % NV;
                        ok = mbar_wait(smem_addr(&sh.v_empty[s]), ((vc / NV) & 1u) ^ 1u, wctx, kSiteLoadKvEmpty);
                        if (!ok) break;
                        const uint32_t bar = smem_addr(&sh.v_full[s]);
                        mbar_arrive_expect_tx(bar, Cfg::kVBytes);
#pragma unroll
                        for (int cc = 0; cc < 2; ++cc)
                            tma_load_4d(sV + s * Cfg::kVBytes + cc * kChunkBytes, &tm_v, bar, cc * kChunkCols,
                                        item.k_row0 + j0, item.kvh, kVarlen ? 0 : item.b);
                        ++vc;
                    }
                }
                // the next item is drawn once the loads of this one are all issued (see fa_fwd_persistent_kernel);
                // the launch makes n_items draws in all, and the CTA that takes the last one zeroes the counter
                const unsigned int ticket = atomicAdd(p.sched_counter, 1u);
                if (ticket == static_cast<unsigned int>(n_items) - 1u) atomicExch(p.sched_counter, 0u);
                idx = G + static_cast<int>(ticket);
            }
        }
    } else if (warp == 10) {
        // ============================================================ TMA loads of the Q tiles
        setmaxnreg_dec<kPairRegsOther>();
        if (elect_one()) {
            uint32_t qc0 = 0, qc1 = 0;       // loads of Q_0 and Q_1 so far
            bool ok = true;
#pragma unroll 1
            for (int k = 0; ok; ++k) {
                if (item_wait_thread(k) < 0) break;
                const PersistItem item = item_at(k);
                item_release_thread(k);
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if ((t == 0 ? item.nkv_0 : item.nkv_1) == 0) continue;
                    const uint32_t qc = (t == 0) ? qc0 : qc1;
                    ok = mbar_wait(smem_addr(&sh.q_empty[t]), (qc & 1u) ^ 1u, wctx, kSiteLoadQEmpty);
                    if (!ok) break;
                    const uint32_t bar = smem_addr(&sh.q_full[t]);
                    mbar_arrive_expect_tx(bar, Cfg::kQBytes);
#pragma unroll
                    for (int cc = 0; cc < 2; ++cc)
                        tma_load_4d(sQ + t * Cfg::kQBytes + cc * kChunkBytes, &tm_q, bar, cc * kChunkCols,
                                    item.q_row0 + (t == 0 ? item.i0_0 : item.i0_1), t == 0 ? item.hq : item.hq1,
                                    kVarlen ? 0 : item.b);
                    if (t == 0) ++qc0; else ++qc1;
                }
            }
        }
    } else {
        setmaxnreg_dec<kPairRegsOther>();     // warp 11: idle, completes the third warpgroup
    }

    // ---------------------------------------------------------------- teardown (all warps)
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem_base, Cfg::kTmemCols);
}

}  // namespace fa
