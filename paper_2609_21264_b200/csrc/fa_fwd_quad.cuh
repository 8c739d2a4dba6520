// Attention forward kernel for sm_100a, head sizes 128 and 192/128: four 128-row query tiles per pair of SMs.
//
// The loop of fa_fwd_pair.cuh (two query tiles per CTA, one softmax warpgroup per tile, P_t over S_t in TMEM, one
// thread that issues every MMA and probes its barriers from inside the blocks of MMAs; read that file first) on a
// cluster of two CTAs with two-CTA MMAs, as fa_fwd_duo.cuh does for one query tile per CTA (read it for the
// cluster protocol).  Accumulator t of CTA 0 and accumulator t of CTA 1 are the two halves of ONE MMA with M = 256:
//     S_t = Q_t K_j^T      A = each CTA's own query tile t, B = K_j: keys [64 r, 64 r + 64) from CTA r
//     O_t += P_t V_j       A = each CTA's own P_t in TMEM,  B = V_j: columns [64 r, 64 r + 64) from CTA r
// so each CTA fetches and keeps HALF of every K/V tile, and its tensor core reads half as many operand bytes
// from shared memory per MMA.  Why that matters: a 128 x 128 x 16 MMA with both operands in shared memory reads
// 8 KB in its 64 cycles, the whole bandwidth of the SM's shared memory, and the TMA writes of the next K/V tiles
// have to fit in beside it; with B halved the score MMAs read 6 KB and the PV MMAs 2 KB, and the shared-memory
// ring holds 5 K/V tiles instead of 2-3 (3 at 192/128).
//
// Which four tiles a cluster takes (kMode), for accumulator t of CTA r:
//   0: one head, four adjacent query tiles: tile 4 g + 2 t + r   (the two halves of an MMA are adjacent tiles)
//   1: two adjacent heads of a K/V group, two adjacent tiles: head h + t, tile 2 g + r
//   2: four adjacent heads of a K/V group, one tile: head h + 2 t + r, tile g   (all four have the same K/V tiles)
// An MMA runs for as many K/V tiles as the longer of its two halves needs; the other half's extra tiles are fully
// masked for it (under a causal mask one tile in mode 0 and 1, none in mode 2).
//
// Roles (384 threads per CTA): warps 0-3 / 4-7 softmax, rescale and epilogue of this CTA's tile 0 / 1; warp 8 MMA
// issue (leader CTA only); warp 9 TMA loads of this CTA's two query tiles and of its halves of K_j, V_j.
// TMEM (each CTA): S_0 [0,128) S_1 [128,256) O_0 [256,384) O_1 [384,512); bf16 P_t overlays S_t[0,64).
// Fixed-length batches without split-KV only.
#pragma once

#include <math.h>

#include "fa_common.cuh"
#include "fa_fwd_duo.cuh"
#include "fa_fwd_pair.cuh"
#include "fa_softmax_pass.cuh"
#include "ptx.cuh"

namespace fa {

namespace ptx {
// Arrive (count 1) on this CTA's barrier only once every tcgen05 operation issued so far by this thread has completed
// (the two-CTA form of the commit; ptx::tc_commit_2cta signals the barrier at the same offset in both CTAs).
FA_DEVI void tc_commit_pair_local(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
}  // namespace ptx

template <int DQK, int DV>
struct QuadCfg {
    static_assert((DQK == 128 || DQK == 192) && DV == 128, "written for head sizes 128/128 and 192/128");
    static constexpr int kQChunks = DQK / kChunkCols;
    static constexpr int kQBytes = kQChunks * kChunkBytes;              // one query tile
    static constexpr int kKHalfChunkBytes = (kTileN / 2) * kChunkCols * 2;   // 64 keys x 64 columns
    static constexpr int kKHalfBytes = kQChunks * kKHalfChunkBytes;     // this CTA's half of a K tile
    static constexpr int kVHalfBytes = kChunkBytes;                     // 128 keys x this CTA's 64 columns of V
    static constexpr int kStages = (DQK == 128) ? 5 : 3;                // of K and of V
    static constexpr int kTileBytes = 2 * kQBytes + kStages * (kKHalfBytes + kVHalfBytes);
    static constexpr int kTmemCols = 512;
    static constexpr int kColS0 = 0, kColS1 = 128, kColO0 = 256, kColO1 = 384;
    static constexpr int kThreads = 384;
    static constexpr int kMaxStages = 5;
};

struct QuadShared {
    uint64_t q_full[2];                   // leader: query tile t of both CTAs has landed
    uint64_t k_full[QuadCfg<128, 128>::kMaxStages], v_full[QuadCfg<128, 128>::kMaxStages];      // leader: both halves have landed
    // each CTA: release r (barrier r mod stages) = the MMAs that read K_r and V_{r-1} are complete.  The MMA thread
    // commits to the leader's barrier only; the leader's loader passes every release on to the partner's barrier.
    uint64_t kv_empty[QuadCfg<128, 128>::kMaxStages];
    uint64_t s_full[2];                   // each CTA: S_t(j) is in TMEM
    uint64_t p_first[2], p_rest[2];       // leader: both CTAs' softmax warps of tile t have written P_t (keys 0..95 / all)
    uint64_t o_final[2];                  // each CTA: the last PV MMA of tile t is complete
    uint64_t o_staged[2];                 // each CTA: the bf16 O_t tile is in shared memory
    uint32_t tmem_base;
    uint32_t abort_flag;
};

template <int DQK, int DV>
constexpr int quad_smem_bytes() {
    return QuadCfg<DQK, DV>::kTileBytes + static_cast<int>(sizeof(QuadShared));
}

template <int DQK, int DV, int kMode>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(384, 1)
fa_fwd_quad_kernel(const __grid_constant__ CUtensorMap tm_q,
                   const __grid_constant__ CUtensorMap tm_k,      // boxes of 64 keys
                   const __grid_constant__ CUtensorMap tm_v,      // boxes of 128 keys x 64 columns
                   const __grid_constant__ CUtensorMap tm_o,
                   const FwdParams p) {
    using Cfg = QuadCfg<DQK, DV>;
    using namespace ptx;
    constexpr int NS = Cfg::kStages;
    constexpr int kKSteps = DQK / 16;
    constexpr int kHeadsPerItem = kMode == 0 ? 1 : (kMode == 1 ? 2 : 4);
    constexpr int kTilesPerHead = 4 / kHeadsPerItem;      // adjacent query tiles of each head

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    QuadShared& sh = *reinterpret_cast<QuadShared*>(smem_raw + Cfg::kTileBytes);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const uint32_t rank = cluster_ctarank();

    grid_launch_dependents();

    const uint32_t smem_base = smem_addr(smem_raw);
    if ((smem_base & 1023u) != 0u) {          // the same in both CTAs of a cluster; nothing has been set up yet
        grid_dependency_wait();
        if (tid == 0 && p.status) {
            volatile uint32_t* sw = p.status;
            sw[1] = kSiteSmemAlign;
            sw[0] = 3u;                       // FA_ERR_CUDA
            __threadfence_system();
        }
        return;
    }
    const uint32_t sQ = smem_base;                                // two tiles
    const uint32_t sK = sQ + 2 * Cfg::kQBytes;                    // NS stages of this CTA's half
    const uint32_t sV = sK + NS * Cfg::kKHalfBytes;               // NS stages of this CTA's half

    // Item decode as in fa_fwd_pair_kernel (L2-sized groups of heads, longest items first), one item per cluster.
    const int n_tg = (p.n_q_tiles + kTilesPerHead - 1) / kTilesPerHead;
    const int n_units = (p.B * p.Hq) / kHeadsPerItem;
    const int hpg = p.heads_per_group / kHeadsPerItem;
    const int item = static_cast<int>(blockIdx.x >> 1);
    const int group = item / (n_tg * hpg);
    const int bh0 = group * hpg;
    const int group_size = (n_units - bh0 < hpg) ? (n_units - bh0) : hpg;
    const int local = item - group * n_tg * hpg;
    const int tg = n_tg - 1 - local / group_size;
    const int bh = kHeadsPerItem * (bh0 + local % group_size);
    const int hq0 = bh % p.Hq;
    const int b = bh / p.Hq;
    const int kvh = hq0 / (p.Hq / p.Hkv);
    const int Sq = p.Sq, Sk = p.Sk;
    const int off = Sk - Sq;

    // accumulator t of CTA r: its head and the first row of its query tile
    auto head_of = [&](int r, int t) -> int { return kMode == 0 ? hq0 : (kMode == 1 ? hq0 + t : hq0 + 2 * t + r); };
    auto row0_of = [&](int r, int t) -> int { return (kMode == 0 ? 4 * tg + 2 * t + r : (kMode == 1 ? 2 * tg + r : tg)) * kTileM; };
    auto tiles_of = [&](int i) -> int { return i < Sq ? kv_tiles_for_q_tile(i, kTileM, Sq, Sk, p.causal) : 0; };
    const int r_own = static_cast<int>(rank);
    const int own_0 = tiles_of(row0_of(r_own, 0)), own_1 = tiles_of(row0_of(r_own, 1));      // this CTA's tiles
    const int oth_0 = tiles_of(row0_of(r_own ^ 1, 0)), oth_1 = tiles_of(row0_of(r_own ^ 1, 1));
    const int nkv_0 = own_0 > oth_0 ? own_0 : oth_0;      // K/V tiles that MMA t runs: the longer of its two halves
    const int nkv_1 = own_1 > oth_1 ? own_1 : oth_1;
    const int n_max = nkv_0 > nkv_1 ? nkv_0 : nkv_1;

    // ---------------------------------------------------------------- setup
    if (tid == 0) {
        sh.abort_flag = 0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_addr(&sh.q_full[t]), 1);
            mbar_init(smem_addr(&sh.s_full[t]), 1);
            mbar_init(smem_addr(&sh.p_first[t]), 8);      // 4 softmax warps of each CTA
            mbar_init(smem_addr(&sh.p_rest[t]), 8);
            mbar_init(smem_addr(&sh.o_final[t]), 1);
            mbar_init(smem_addr(&sh.o_staged[t]), 4);
        }
#pragma unroll
        for (int s = 0; s < Cfg::kMaxStages; ++s) {
            mbar_init(smem_addr(&sh.k_full[s]), 1);
            mbar_init(smem_addr(&sh.v_full[s]), 1);
            mbar_init(smem_addr(&sh.kv_empty[s]), 1);
        }
        fence_mbar_init();
    }
    if (warp == 8) {
        tmem_alloc_2cta(smem_addr(&sh.tmem_base), Cfg::kTmemCols);
        tmem_relinquish_alloc_permit_2cta();
    }
    if (warp == 9 && lane == 0) {
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
        prefetch_tensormap(&tm_o);
    }
    tc_fence_before_sync();
    __syncthreads();
    // the partner's barriers are initialised before anything of this CTA can reach them
    cluster_arrive_release();
    cluster_wait_acquire();
    tc_fence_after_sync();
    grid_dependency_wait();

    const uint32_t tmem_base = sh.tmem_base;
    DuoWaitCtx wctx{&sh.abort_flag, mapa_shared(smem_addr(&sh.abort_flag), rank ^ 1u), p.status, p.wait_limit_ns};
    const float c = p.scale_log2;

    if (warp < 8) {
        // ============================================================ softmax of this CTA's tile t
        setmaxnreg_inc<kPairRegsSoftmax>();
        const int t = warp >> 2;
        const int row = tid & (kTileM - 1);
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + (t == 0 ? Cfg::kColS0 : Cfg::kColS1) + lane_sel;
        const uint32_t tO = tmem_base + (t == 0 ? Cfg::kColO0 : Cfg::kColO1) + lane_sel;
        const uint32_t bar_s = smem_addr(&sh.s_full[t]);
        const uint32_t bar_pf = mapa_shared(smem_addr(&sh.p_first[t]), 0u);    // the leader's
        const uint32_t bar_pr = mapa_shared(smem_addr(&sh.p_rest[t]), 0u);
        const int i0_t = row0_of(r_own, t);
        const int hq_t = head_of(r_own, t);
        const int q_idx_t = b * p.Hq + hq_t;
        const int nkv_t = t == 0 ? nkv_0 : nkv_1;        // passes (the MMA's count)
        const int own_t = t == 0 ? own_0 : own_1;        // K/V tiles with a visible key for this tile
        const int i_glob = i0_t + row;
        int kmax_row = Sk - 1;
        if (p.causal && i_glob + off < kmax_row) kmax_row = i_glob + off;
        const float tau_raw = kRescaleThresholdLog2 / c;

        float m_ref = -INFINITY;   // reference maximum, raw score units
        float l = 0.f;
        bool ok = true;
        FA_PHASE_DECL();      // phases: 0 wait for S, 5 the pass
        for (int j = 0; j < nkv_t; ++j) {
            ok = __all_sync(0xffffffffu, duo_wait<false>(bar_s, j & 1, wctx, kSiteSoftmaxSFull));
            if (!ok) break;
            tc_fence_after_sync();
            FA_PHASE(0);
            softmax_pass_128<DV>(tS, tO, c, tau_raw, j * kTileN, kmax_row, j == 0, m_ref, l, lane,
                                 [&]() { mbar_arrive_cluster(bar_pf); }, [&]() { mbar_arrive_cluster(bar_pr); });
            FA_PHASE(5);
        }
        FA_PHASE_STORE(6, nkv_t);
        // epilogue: O = G' / s (bf16), lse = u * scale + ln s   (as in fa_fwd_pair_kernel)
        if (ok && i0_t < Sq) {
            const size_t lse_row0 = static_cast<size_t>(q_idx_t) * p.Sq;
            __nv_bfloat16* o_row = p.O + (b * p.o_stride_b + hq_t * p.o_stride_h + static_cast<long long>(i_glob) * p.o_stride_s);
            if (own_t == 0) {         // no key visible to any row of this tile
                if (i_glob < Sq) {
                    const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int v = 0; v < DV / 8; ++v) reinterpret_cast<uint4*>(o_row)[v] = z;
                    if (p.lse) p.lse[lse_row0 + i_glob] = -INFINITY;
                }
            } else if (__all_sync(0xffffffffu, duo_wait<false>(smem_addr(&sh.o_final[t]), 0, wctx, kSiteEpiOFull))) {
                tc_fence_after_sync();
                const float inv_l = (l > 0.f) ? (1.f / l) : 0.f;
                if (p.lse && i_glob < Sq)
                    p.lse[lse_row0 + i_glob] = (l > 0.f) ? (m_ref * c * 0.6931471805599453f + logf(l)) : -INFINITY;
                // staged in the Q tile's space (its last reader, the final score MMA, is complete)
                const uint32_t sO = sQ + t * Cfg::kQBytes + row * 128;
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
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_addr(&sh.o_staged[t]));
                if ((warp & 3) == 0 && lane == 0 &&
                    duo_wait<false>(smem_addr(&sh.o_staged[t]), 0, wctx, kSiteEpiStaged)) {
#pragma unroll
                    for (int ch = 0; ch < DV / kChunkCols; ++ch)
                        tma_store_4d(&tm_o, sQ + t * Cfg::kQBytes + ch * kChunkBytes, ch * kChunkCols, i0_t, hq_t, b);
                    tma_store_commit();
                    tma_store_wait_read_all();     // the CTA's shared memory outlives the reads
                }
            }
        }
    } else if (warp == 8) {
        // ============================================================ MMA issue: one thread of the leader CTA
        setmaxnreg_dec<kPairRegsOther>();
        if (rank == 0 && elect_one() && n_max > 0) {
            constexpr uint32_t kIdescQK = make_idesc_bf16_f32(2 * kTileM, kTileN, false, false);
            constexpr uint32_t kIdescPV = make_idesc_bf16_f32(2 * kTileM, DV, false, true);
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // sbo, version, swizzle
            const uint32_t q_lo0 = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t v_lo0 = ((sV & 0x3FFFFu) >> 4) | ((static_cast<uint32_t>(kChunkBytes) >> 4) << 16);
            auto desc = [](uint32_t lo) -> uint64_t {
                return (static_cast<uint64_t>(kDescHi) << 32) | lo;
            };
            // k-step k of a query tile (chunks of 128 rows) and of this CTA's half of K (chunks of 64 rows)
            auto qoff = [](int k) -> uint32_t { return static_cast<uint32_t>(((k / 4) * kChunkBytes + (k % 4) * 32) >> 4); };
            auto koff = [](int k) -> uint32_t { return static_cast<uint32_t>(((k / 4) * Cfg::kKHalfChunkBytes + (k % 4) * 32) >> 4); };
            auto commit_all = [](uint32_t bar) { tc_commit_2cta(bar, mapa_shared(bar, 1u)); };
            // a barrier whose phase 0 completed long ago and which never moves again: filler for unused probe slots
            const uint32_t bar_always = smem_addr(&sh.q_full[nkv_0 > 0 ? 0 : 1]);

            bool ok = duo_wait<false>(smem_addr(&sh.k_full[0]), 0, wctx, kSiteMmaKvFull);
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (ok && (t == 0 ? nkv_0 : nkv_1) > 0) {
                    ok = duo_wait<false>(smem_addr(&sh.q_full[t]), 0, wctx, kSiteMmaQFull);
                    if (ok) {
                        tc_fence_after_sync();
                        const uint32_t tS = tmem_base + (t == 0 ? Cfg::kColS0 : Cfg::kColS1);
                        const uint32_t q_lo = q_lo0 + t * (Cfg::kQBytes >> 4);
#pragma unroll
                        for (int k = 0; k < kKSteps; ++k)
                            mma2_ss(tS, desc(q_lo + qoff(k)), desc(k_lo0 + koff(k)), kIdescQK, k > 0 ? 1u : 0u);
                        commit_all(smem_addr(&sh.s_full[t]));
                    }
                }
            }
            if (ok) tc_commit_pair_local(smem_addr(&sh.kv_empty[0]));      // release 0: K_0
            int sv = 0, sk = 1;                      // stage of V_j and of K_{j+1}
            uint32_t ph_v = 0, ph_k = 0;
            // results of the probes made from inside the block before: P_0 / P_1 first part, V_j, K_{j+1}
            uint32_t pre_p0 = 0u, pre_p1 = 0u, pre_v = 0u, pre_k = 0u;
            FA_PHASE_DECL();      // phases: 0 K/V ring and commits, 1 wait for P (first part), 2 first MMAs, 3 wait for P (rest), 4 other MMAs

            // One tile's block of iteration j: PV_t(j), then QK_t(j+1).  (b0, par0) ... (b2, par2): barriers to
            // probe from inside the block; the result lands in `probed` (bit i = probe i succeeded).
            auto tile_block = [&](auto tc, int j, int nkv_t, uint32_t pre_first, uint32_t b0, uint32_t par0, uint32_t b1,
                                  uint32_t par1, uint32_t b2, uint32_t par2, uint32_t& probed) -> bool {
                constexpr int t = decltype(tc)::value;
                probed = 0u;
                if (j >= nkv_t) return true;
                const uint32_t tS = tmem_base + (t == 0 ? Cfg::kColS0 : Cfg::kColS1);   // P_t overlays it
                const uint32_t tO = tmem_base + (t == 0 ? Cfg::kColO0 : Cfg::kColO1);
                const uint32_t q_lo = q_lo0 + t * (Cfg::kQBytes >> 4);
                const uint32_t vlo = v_lo0 + sv * (Cfg::kVHalfBytes >> 4);
                const uint32_t klo = k_lo0 + sk * (Cfg::kKHalfBytes >> 4);
                FA_PHASE(0);
                if (!pre_first && !duo_wait<true>(smem_addr(&sh.p_first[t]), j & 1, wctx, kSiteMmaPFull)) return false;
                FA_PHASE(1);
                tc_fence_after_sync();
                // PV k-steps 0..3, then the probe of p_rest under k-steps 4 and 5
                mma2_ts(tO, tS + 0, desc(vlo + 0 * (2048 >> 4)), kIdescPV, j > 0 ? 1u : 0u);
                mma2_ts(tO, tS + 8, desc(vlo + 1 * (2048 >> 4)), kIdescPV, 1u);
                mma2_ts(tO, tS + 16, desc(vlo + 2 * (2048 >> 4)), kIdescPV, 1u);
                mma2_ts(tO, tS + 24, desc(vlo + 3 * (2048 >> 4)), kIdescPV, 1u);
                const uint32_t rest = probe_mma2_ts2(smem_addr(&sh.p_rest[t]), j & 1, tO, tS + 32, desc(vlo + 4 * (2048 >> 4)),
                                                     tS + 40, desc(vlo + 5 * (2048 >> 4)), kIdescPV);
                FA_PHASE(2);
                if (!rest && !duo_wait<true>(smem_addr(&sh.p_rest[t]), j & 1, wctx, kSiteMmaPFull)) return false;
                FA_PHASE(3);
                tc_fence_after_sync();
                mma2_ts(tO, tS + 48, desc(vlo + 6 * (2048 >> 4)), kIdescPV, 1u);
                mma2_ts(tO, tS + 56, desc(vlo + 7 * (2048 >> 4)), kIdescPV, 1u);
                if (j + 1 < nkv_t) {
                    mma2_ss(tS, desc(q_lo + qoff(0)), desc(klo + koff(0)), kIdescQK, 0u);
                    mma2_ss(tS, desc(q_lo + qoff(1)), desc(klo + koff(1)), kIdescQK, 1u);
                    mma2_ss(tS, desc(q_lo + qoff(2)), desc(klo + koff(2)), kIdescQK, 1u);
                    mma2_ss(tS, desc(q_lo + qoff(3)), desc(klo + koff(3)), kIdescQK, 1u);
                    probed = probe3_mma2_ss3(b0, par0, b1, par1, b2, par2, tS, desc(q_lo + qoff(4)), desc(klo + koff(4)),
                                             desc(q_lo + qoff(5)), desc(klo + koff(5)), desc(q_lo + qoff(6)), desc(klo + koff(6)),
                                             kIdescQK);
#pragma unroll
                    for (int k = 7; k < kKSteps; ++k)
                        mma2_ss(tS, desc(q_lo + qoff(k)), desc(klo + koff(k)), kIdescQK, 1u);
                    commit_all(smem_addr(&sh.s_full[t]));
                } else {
                    commit_all(smem_addr(&sh.o_final[t]));
                }
                FA_PHASE(4);
                return true;
            };

            for (int j = 0; j < n_max && ok; ++j) {
                if (!pre_v) ok = duo_wait<false>(smem_addr(&sh.v_full[sv]), ph_v, wctx, kSiteMmaKvFull);
                if (ok && j + 1 < n_max && !pre_k) ok = duo_wait<false>(smem_addr(&sh.k_full[sk]), ph_k, wctx, kSiteMmaKvFull);
                if (!ok) break;
                FA_PHASE(5);
                uint32_t probed;
                // block of tile 0; probes: first part of P_1(j)
                ok = tile_block(IntC<0>{}, j, nkv_0, pre_p0, (j < nkv_1) ? smem_addr(&sh.p_first[1]) : bar_always,
                                (j < nkv_1) ? (j & 1) : 0u, bar_always, 0u, bar_always, 0u, probed);
                if (!ok) break;
                pre_p1 = (j < nkv_1) ? (probed & 1u) : 0u;
                // stage and phase of V_{j+1} and K_{j+2}
                int sv_n = sv + 1; uint32_t ph_v_n = ph_v; if (sv_n == NS) { sv_n = 0; ph_v_n ^= 1u; }
                int sk_n = sk + 1; uint32_t ph_k_n = ph_k; if (sk_n == NS) { sk_n = 0; ph_k_n ^= 1u; }
                // block of tile 1; probes: first part of P_0(j+1), V_{j+1}, K_{j+2}
                const bool next_p0 = j + 1 < nkv_0, next_v = j + 1 < n_max, next_k = j + 2 < n_max;
                ok = tile_block(IntC<1>{}, j, nkv_1, pre_p1,
                                next_p0 ? smem_addr(&sh.p_first[0]) : bar_always, next_p0 ? ((j + 1) & 1) : 0u,
                                next_v ? smem_addr(&sh.v_full[sv_n]) : bar_always, next_v ? ph_v_n : 0u,
                                next_k ? smem_addr(&sh.k_full[sk_n]) : bar_always, next_k ? ph_k_n : 0u, probed);
                if (!ok) break;
                pre_p0 = next_p0 ? (probed & 1u) : 0u;
                pre_v = next_v ? ((probed >> 1) & 1u) : 0u;
                pre_k = next_k ? ((probed >> 2) & 1u) : 0u;
                tc_commit_pair_local(smem_addr(&sh.kv_empty[sk]));        // release j + 1: V_j and K_{j+1} (stage (j + 1) mod NS)
                FA_PHASE(6);
                sv = sv_n; ph_v = ph_v_n; sk = sk_n; ph_k = ph_k_n;
            }
            FA_PHASE_STORE(7, n_max);
        }
    } else if (warp == 9) {
        // ============================================================ TMA loads: this CTA's query tiles and its halves of K_j, V_j
        setmaxnreg_dec<kPairRegsOther>();
        if (elect_one() && n_max > 0) {
            auto load_q = [&](int t) {
                if ((t == 0 ? nkv_0 : nkv_1) == 0) return;
                if (rank == 0) mbar_arrive_expect_tx(smem_addr(&sh.q_full[t]), 2 * Cfg::kQBytes);
                const uint32_t bar = mapa_shared(smem_addr(&sh.q_full[t]), 0u);
#pragma unroll
                for (int cc = 0; cc < Cfg::kQChunks; ++cc)
                    tma_load_4d_2cta(sQ + t * Cfg::kQBytes + cc * kChunkBytes, &tm_q, bar, cc * kChunkCols, row0_of(r_own, t),
                                     head_of(r_own, t), b);
            };
            load_q(0);
            bool ok = true;
            FA_PHASE_DECL();      // phases: 0 issue, 2 wait for a release
            for (int j = 0; j < n_max && ok; ++j) {
                const int j0 = j * kTileN;
                const int s = j % NS;
                {
                    // K_j: its stage held K_{j-NS}, freed by release j - NS, which step j - 1 waited for
                    if (rank == 0) mbar_arrive_expect_tx(smem_addr(&sh.k_full[s]), 2 * Cfg::kKHalfBytes);
                    const uint32_t bar = mapa_shared(smem_addr(&sh.k_full[s]), 0u);
#pragma unroll
                    for (int cc = 0; cc < Cfg::kQChunks; ++cc)
                        tma_load_4d_2cta(sK + s * Cfg::kKHalfBytes + cc * Cfg::kKHalfChunkBytes, &tm_k, bar, cc * kChunkCols,
                                         j0 + r_own * (kTileN / 2), kvh, b);
                    if (j == 0) load_q(1);
                }
                // V_j: its stage held V_{j-NS}, freed by release r = j - NS + 1 (which also frees the stage of K_{j+1})
                const int r = j - NS + 1;
                if (r >= 0) {
                    const uint32_t bar_e = smem_addr(&sh.kv_empty[r % NS]);
                    FA_PHASE(0);
                    ok = duo_wait<false>(bar_e, (r / NS) & 1, wctx, kSiteLoadKvEmpty);
                    FA_PHASE(2);
                    if (!ok) break;
                    if (rank == 0) mbar_arrive_cluster(mapa_shared(bar_e, 1u));     // pass it on to the partner's loader
                }
                if (!(p.debug_drop_v_load && j == 0)) {
                    if (rank == 0) mbar_arrive_expect_tx(smem_addr(&sh.v_full[s]), 2 * Cfg::kVHalfBytes);
                    const uint32_t bar = mapa_shared(smem_addr(&sh.v_full[s]), 0u);
                    tma_load_4d_2cta(sV + s * Cfg::kVHalfBytes, &tm_v, bar, r_own * kChunkCols, j0, kvh, b);
                }
            }
            FA_PHASE_STORE(3, n_max);
        }
    } else {
        setmaxnreg_dec<kPairRegsOther>();     // idle warps of the third warpgroup
    }

    // ---------------------------------------------------------------- teardown (all warps of both CTAs)
    tc_fence_before_sync();
    __syncthreads();
    cluster_arrive_release();
    cluster_wait_acquire();
    if (warp == 8) tmem_dealloc_2cta(tmem_base, Cfg::kTmemCols);
}

}  // namespace fa
