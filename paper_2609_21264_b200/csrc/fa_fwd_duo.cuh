// Attention forward kernel for sm_100a on pairs of SMs: a cluster of two CTAs, one 128-row query tile per
// CTA, every MMA issued once for both as a 256-row tcgen05.mma.cta_group::2.  Head sizes 128/128 and 192/128.
//
// Why.  With one CTA per SM every CTA streams whole K/V tiles from L2 into its own shared memory.  At head
// sizes 192/128 a K tile is 48 KB and a V tile 32 KB; next to Q (48 KB) only two stages of each fit, and a
// ring of two does not cover the latency of its own refill (measured: the tensor pipe is about 50 % busy on
// such shapes with one tile per CTA, and two query tiles per CTA leave room for even fewer stages).  A CTA
// pair splits every K/V tile: CTA r keeps keys [64r, 64r+64) of K_j (the N dimension of S = Q K^T) and
// columns [64r, 64r+64) of V_j (the N dimension of O += P V), and the two-CTA MMA reads both halves.  That
// halves the L2 -> shared memory traffic per query tile and doubles the ring depth (4 + 4 stages) in the
// same shared memory.
//
// The loop is the one of fa_fwd_pair.cuh (read that file first: one elected MMA thread, barrier probes
// inside blocks of MMAs, no correction warps, P handed over in two parts), applied to the even and the odd
// K/V tiles of ONE query tile instead of to two query tiles: score buffer b and accumulator O^b belong to
// the K/V tiles j = b, b+2, b+4, ..., softmax warpgroup b keeps its own reference maximum and row sum for
// them, and the two partial results are merged once, in the epilogue, with the split/merge identity of the
// online softmax (Algorithm 2's merge in its corrected form):
//     u = max(u_0, u_1),  s = s_0 2^(u_0-u) + s_1 2^(u_1-u),  O = (O^0 2^(u_0-u) + O^1 2^(u_1-u)) / s.
// So the summation order differs from the other kernels': results agree with them to rounding, not bit for bit.
//
// Cluster protocol (rank 0 = leader; only its warp 8 issues MMAs):
//   q_full, k_full[], v_full[], p_first[], p_rest[]   live in the leader: TMA loads of both CTAs complete
//       their bytes there (cp.async.bulk.tensor with .cta_group::2), softmax warps of both CTAs arrive there
//       (mbarrier.arrive on the mapped shared::cluster address);
//   s_full[], k_empty[], v_empty[], o_final            exist in both CTAs and are signalled in both by a pair of
//       tcgen05.commit.cta_group::2, one per CTA (the partner's barrier through its mapped address);
//   every wait is bounded as elsewhere; a wait that runs out raises the abort flag of both CTAs.
// A CTA must not exit while its partner can still touch its shared memory or TMEM: all threads of the
// cluster meet at a cluster barrier before TMEM is freed.  (barrier.cluster.wait only waits for threads
// that have not exited, so a CTA that returned early cannot hang its partner.)
//
// Roles (384 threads per CTA): warps 0-3 / 4-7 softmax of the even / odd K/V tiles, warp 8 MMA issue
// (leader) and TMEM allocation (both), warp 9 TMA loads, warps 10-11 idle.
// TMEM (per CTA): S^0 [0,128) S^1 [128,256) O^0 [256,384) O^1 [384,512); bf16 P^b overlays S^b[0,64).
#pragma once

#include <math.h>

#include "fa_common.cuh"
#include "fa_fwd_pair.cuh"
#include "ptx.cuh"

namespace fa {

template <int DQK, int DV>
struct DuoCfg {
    static_assert((DQK == 128 || DQK == 192) && DV == 128, "the two-CTA kernel is written for head sizes 128/128 and 192/128");
    static constexpr int kQChunks = DQK / kChunkCols;
    static constexpr int kQBytes = kQChunks * kChunkBytes;          // one query tile
    static constexpr int kKHalfChunkBytes = (kTileN / 2) * kChunkCols * 2;   // 64 keys x 64 columns = 8 KB
    static constexpr int kKHalfBytes = kQChunks * kKHalfChunkBytes;  // this CTA's 64 keys of a K tile
    static constexpr int kVHalfBytes = kChunkBytes;                  // this CTA's 64 columns of a V tile (128 keys)
    static constexpr int kKStages = 4;
    static constexpr int kVStages = 4;
    static constexpr int kTileBytes = kQBytes + kKStages * kKHalfBytes + kVStages * kVHalfBytes;
    static constexpr int kTmemCols = 512;
    static constexpr int kColS0 = 0, kColS1 = 128, kColO0 = 256, kColO1 = 384;
    static constexpr int kThreads = 384;
};

struct DuoShared {
    uint64_t q_full;                      // leader: Q of both CTAs has landed
    uint64_t k_full[4], v_full[4];        // leader: both halves of the stage have landed
    uint64_t k_empty[4], v_empty[4];      // each CTA: the MMAs that read the stage are complete
    uint64_t s_full[2];                   // each CTA: S^b(j) is in TMEM
    uint64_t p_first[2], p_rest[2];       // leader: both CTAs' softmax warps have written P^b (keys 0..95 / all)
    uint64_t o_final;                     // each CTA: every MMA is complete
    uint64_t st_ready;                    // each CTA: both warpgroups' row state is in `state`
    uint64_t o_staged[2];                 // each CTA: half b of the bf16 O tile is in shared memory
    float2 state[2][kTileM];              // (reference maximum in log2 units, row sum) of warpgroup b
    uint32_t tmem_base;
    uint32_t abort_flag;
};

template <int DQK, int DV>
constexpr int duo_smem_bytes() {
    return DuoCfg<DQK, DV>::kTileBytes + static_cast<int>(sizeof(DuoShared));
}

struct DuoWaitCtx {
    volatile uint32_t* abort_flag;    // this CTA's
    uint32_t peer_abort;              // shared::cluster address of the partner's
    uint32_t* status;
    uint64_t limit_ns;
};

// Bounded wait, as ptx::mbar_wait (kCluster only marks the waits whose phase the partner CTA's arrivals complete).
// Giving up raises the abort flag of both CTAs.
template <bool kCluster>
FA_DEVI bool duo_wait(uint32_t bar, uint32_t parity, const DuoWaitCtx& ctx, uint32_t who) {
    auto probe = [&]() { return ptx::mbar_try_wait(bar, parity); };
    if (probe()) return true;
    uint64_t t0 = 0;
    for (uint32_t it = 1;; ++it) {
        if (probe()) return true;
        if ((it & 63u) == 0u) {
            if (*ctx.abort_flag) return false;
            const uint64_t now = ptx::globaltimer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > ctx.limit_ns) {
                *ctx.abort_flag = 1u;
                ptx::st_shared_cluster_u32(ctx.peer_abort, 1u);
                if (ctx.status) {
                    volatile uint32_t* sw = ctx.status;
                    sw[1] = who;
                    sw[0] = 4u;                           // FA_ERR_DEVICE_TIMEOUT
                    __threadfence_system();
                }
                return false;
            }
        }
    }
}

// kHeadPair: the two CTAs take the same query tile of two adjacent heads of a K/V group (causal grouped
// heads: both see the same K/V tiles); otherwise two adjacent query tiles of one head.
template <int DQK, int DV, bool kHeadPair = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(384, 1)
fa_fwd_duo_kernel(const __grid_constant__ CUtensorMap tm_q,
                  const __grid_constant__ CUtensorMap tm_k,      // boxes of 64 keys
                  const __grid_constant__ CUtensorMap tm_v,      // boxes of 128 keys
                  const __grid_constant__ CUtensorMap tm_o,
                  const FwdParams p) {
    using Cfg = DuoCfg<DQK, DV>;
    using namespace ptx;
    constexpr int NK = Cfg::kKStages;
    constexpr int NV = Cfg::kVStages;
    constexpr int kKSteps = DQK / 16;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    DuoShared& sh = *reinterpret_cast<DuoShared*>(smem_raw + Cfg::kTileBytes);

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
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + Cfg::kQBytes;                       // NK stages of this CTA's half
    const uint32_t sV = sK + NK * Cfg::kKHalfBytes;              // NV stages of this CTA's half

    // Item decode as in fa_fwd_pair_kernel, one item per cluster.
    const int n_pairs = kHeadPair ? p.n_q_tiles : (p.n_q_tiles + 1) / 2;
    const int n_bh = p.B * p.Hq;
    const int item = static_cast<int>(blockIdx.x >> 1);
    const int hpg = kHeadPair ? p.heads_per_group / 2 : p.heads_per_group;
    const int n_units = kHeadPair ? n_bh / 2 : n_bh;
    const int group = item / (n_pairs * hpg);
    const int bh0 = group * hpg;
    const int group_size = (n_units - bh0 < hpg) ? (n_units - bh0) : hpg;
    const int local = item - group * n_pairs * hpg;
    const int pair = n_pairs - 1 - local / group_size;
    const int bh = kHeadPair ? 2 * (bh0 + local % group_size) : bh0 + local % group_size;
    const int hq0 = bh % p.Hq;
    const int b = bh / p.Hq;
    const int kvh = hq0 / (p.Hq / p.Hkv);
    const int Sq = p.Sq, Sk = p.Sk;
    const int off = Sk - Sq;

    // this CTA's query tile, and the partner's (for the common loop count)
    const int hq = kHeadPair ? hq0 + static_cast<int>(rank) : hq0;
    const int q_idx = b * p.Hq + hq;
    const int i0_r0 = (kHeadPair ? pair : 2 * pair) * kTileM;
    const int i0_r1 = kHeadPair ? i0_r0 : i0_r0 + kTileM;
    const int i0 = rank == 0 ? i0_r0 : i0_r1;
    auto tiles_of = [&](int i) -> int { return i < Sq ? kv_tiles_for_q_tile(i, kTileM, Sq, Sk, p.causal) : 0; };
    const int n_r0 = tiles_of(i0_r0), n_r1 = tiles_of(i0_r1);
    const int n_kv = n_r0 > n_r1 ? n_r0 : n_r1;           // K/V tiles the cluster runs; tiles past a CTA's own count are fully masked for it
    const int nkv_0 = (n_kv + 1) >> 1, nkv_1 = n_kv >> 1;   // tiles of score buffer 0 / 1

    // ---------------------------------------------------------------- setup
    if (tid == 0) {
        sh.abort_flag = 0;
        mbar_init(smem_addr(&sh.q_full), 1);
        mbar_init(smem_addr(&sh.o_final), 1);
        mbar_init(smem_addr(&sh.st_ready), 8);
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_addr(&sh.s_full[t]), 1);
            mbar_init(smem_addr(&sh.p_first[t]), 8);      // 4 softmax warps of each CTA
            mbar_init(smem_addr(&sh.p_rest[t]), 8);
            mbar_init(smem_addr(&sh.o_staged[t]), 4);
        }
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            mbar_init(smem_addr(&sh.k_full[s]), 1);
            mbar_init(smem_addr(&sh.k_empty[s]), 1);
            mbar_init(smem_addr(&sh.v_full[s]), 1);
            mbar_init(smem_addr(&sh.v_empty[s]), 1);
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
        // ============================================================ softmax of the K/V tiles j = wg, wg+2, ...
        setmaxnreg_inc<kPairRegsSoftmax>();
        const int wg = warp >> 2;
        const int row = tid & (kTileM - 1);
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + (wg == 0 ? Cfg::kColS0 : Cfg::kColS1) + lane_sel;
        const uint32_t tO = tmem_base + (wg == 0 ? Cfg::kColO0 : Cfg::kColO1) + lane_sel;
        const uint32_t bar_s = smem_addr(&sh.s_full[wg]);
        const uint32_t bar_pf = mapa_shared(smem_addr(&sh.p_first[wg]), 0u);    // the leader's
        const uint32_t bar_pr = mapa_shared(smem_addr(&sh.p_rest[wg]), 0u);
        const int nkv_w = wg == 0 ? nkv_0 : nkv_1;
        const int i_glob = i0 + row;
        int kmax_row = Sk - 1;
        if (p.causal && i_glob + off < kmax_row) kmax_row = i_glob + off;
        const float tau_raw = kRescaleThresholdLog2 / c;

        float m_ref = -INFINITY;   // reference maximum, raw score units
        float l = 0.f;
        bool ok = true;
        for (int i = 0; i < nkv_w; ++i) {
            ok = __all_sync(0xffffffffu, duo_wait<false>(bar_s, i & 1, wctx, kSiteSoftmaxSFull));
            if (!ok) break;
            tc_fence_after_sync();
            softmax_pass_128<DV>(tS, tO, c, tau_raw, (2 * i + wg) * kTileN, kmax_row, i == 0, m_ref, l, lane,
                                 [&]() { mbar_arrive_cluster(bar_pf); }, [&]() { mbar_arrive_cluster(bar_pr); });
        }

        // ---- epilogue: merge the two warpgroups' partial results, O = (O^0 f_0 + O^1 f_1) / s
        if (ok && i0 < Sq) {
            const size_t lse_row0 = static_cast<size_t>(q_idx) * p.Sq;
            __nv_bfloat16* o_row = p.O + (b * p.o_stride_b + hq * p.o_stride_h + static_cast<long long>(i_glob) * p.o_stride_s);
            if (n_kv == 0) {          // no key visible to any row of the cluster's tiles
                if (wg == 0 && i_glob < Sq) {
                    const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int v = 0; v < DV / 8; ++v) reinterpret_cast<uint4*>(o_row)[v] = z;
                    if (p.lse) p.lse[lse_row0 + i_glob] = -INFINITY;
                }
            } else {
                sh.state[wg][row] = make_float2(m_ref == -INFINITY ? -INFINITY : m_ref * c, l);
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_addr(&sh.st_ready));
                bool go = __all_sync(0xffffffffu, duo_wait<false>(smem_addr(&sh.st_ready), 0, wctx, kSiteEpiState));
                if (go) go = __all_sync(0xffffffffu, duo_wait<false>(smem_addr(&sh.o_final), 0, wctx, kSiteEpiOFull));
                if (go) {
                    tc_fence_after_sync();
                    const float2 st0 = sh.state[0][row], st1 = sh.state[1][row];
                    const float u = fmaxf(st0.x, st1.x);
                    float f0 = 0.f, f1 = 0.f, ssum = 0.f;
                    if (u != -INFINITY) {
                        f0 = exp2_approx(st0.x - u);      // 2^(-inf) = 0 for a warpgroup that saw no visible key
                        f1 = (nkv_1 > 0) ? exp2_approx(st1.x - u) : 0.f;
                        ssum = st0.y * f0 + st1.y * f1;
                    }
                    const float inv = ssum > 0.f ? 1.f / ssum : 0.f;
                    f0 *= inv;
                    f1 *= inv;
                    if (wg == 0 && p.lse && i_glob < Sq)
                        p.lse[lse_row0 + i_glob] = ssum > 0.f ? (u * 0.6931471805599453f + logf(ssum)) : -INFINITY;
                    // warpgroup wg merges columns [64 wg, 64 wg + 64) and stages them as chunk wg of the bf16 tile in
                    // the Q tile's space (its last reader, the final score MMA, is complete)
                    const uint32_t tO0 = tmem_base + Cfg::kColO0 + lane_sel + wg * 64;
                    const uint32_t tO1 = tmem_base + Cfg::kColO1 + lane_sel + wg * 64;
                    const uint32_t chunk = sQ + wg * kChunkBytes + row * 128;
#pragma unroll 1
                    for (int cc = 0; cc < 2; ++cc) {
                        uint32_t r0[32], r1[32];
                        tmem_ld_x32(tO0 + cc * 32, r0);
                        if (nkv_1 > 0) tmem_ld_x32(tO1 + cc * 32, r1);
                        tc_wait_ld();
                        float o[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) {
                            o[e] = __uint_as_float(r0[e]) * f0;
                            if (nkv_1 > 0) o[e] = fmaf(__uint_as_float(r1[e]), f1, o[e]);
                        }
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            const uint32_t piece = static_cast<uint32_t>((cc * 4 + v) ^ (row & 7)) << 4;
                            st_shared_v4(chunk + piece, pack_bf16x2(o[8 * v], o[8 * v + 1]), pack_bf16x2(o[8 * v + 2], o[8 * v + 3]),
                                         pack_bf16x2(o[8 * v + 4], o[8 * v + 5]), pack_bf16x2(o[8 * v + 6], o[8 * v + 7]));
                        }
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_addr(&sh.o_staged[wg]));
                    if ((warp & 3) == 0 && lane == 0 &&
                        duo_wait<false>(smem_addr(&sh.o_staged[wg]), 0, wctx, kSiteEpiStaged)) {
                        tma_store_4d(&tm_o, sQ + wg * kChunkBytes, wg * kChunkCols, i0, hq, b);
                        tma_store_commit();
                        tma_store_wait_read_all();     // the CTA's shared memory outlives the reads
                    }
                }
            }
        }
    } else if (warp == 8) {
        // ============================================================ MMA issue: one thread of the leader CTA
        setmaxnreg_dec<kPairRegsOther>();
        if (rank == 0 && elect_one() && n_kv > 0) {
            constexpr uint32_t kIdescQK = make_idesc_bf16_f32(2 * kTileM, kTileN, false, false);
            constexpr uint32_t kIdescPV = make_idesc_bf16_f32(2 * kTileM, DV, false, true);
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // sbo, version, swizzle
            const uint32_t q_lo = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t v_lo0 = ((sV & 0x3FFFFu) >> 4) | ((static_cast<uint32_t>(kChunkBytes) >> 4) << 16);
            auto desc = [](uint32_t lo) -> uint64_t {
                return (static_cast<uint64_t>(kDescHi) << 32) | lo;
            };
            // k-step k of Q (chunks of 128 rows) and of this CTA's half of K (chunks of 64 rows)
            auto qoff = [](int k) -> uint32_t { return static_cast<uint32_t>(((k / 4) * kChunkBytes + (k % 4) * 32) >> 4); };
            auto koff = [](int k) -> uint32_t { return static_cast<uint32_t>(((k / 4) * Cfg::kKHalfChunkBytes + (k % 4) * 32) >> 4); };
            // a barrier whose phase 0 completed long ago and which never moves again: filler for unused probe slots
            const uint32_t bar_always = smem_addr(&sh.q_full);

            bool ok = duo_wait<false>(smem_addr(&sh.q_full), 0, wctx, kSiteMmaQFull);
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (ok && t < n_kv) {
                    ok = duo_wait<false>(smem_addr(&sh.k_full[t]), 0, wctx, kSiteMmaKvFull);
                    if (ok) {
                        tc_fence_after_sync();
                        const uint32_t tS = tmem_base + (t == 0 ? Cfg::kColS0 : Cfg::kColS1);
                        const uint32_t klo = k_lo0 + t * (Cfg::kKHalfBytes >> 4);
#pragma unroll
                        for (int k = 0; k < kKSteps; ++k)
                            mma2_ss(tS, desc(q_lo + qoff(k)), desc(klo + koff(k)), kIdescQK, k > 0 ? 1u : 0u);
                        tc_commit_2cta(smem_addr(&sh.s_full[t]), mapa_shared(smem_addr(&sh.s_full[t]), 1u));
                        tc_commit_2cta(smem_addr(&sh.k_empty[t]), mapa_shared(smem_addr(&sh.k_empty[t]), 1u));
                    }
                }
            }
            int sv = 0, sk = 2 % NK;              // stage of V_j and of K_{j+2}
            uint32_t ph_v = 0, ph_k = (2 / NK) & 1;
            // results of the probes made from inside the block before: P(j) first part, V_j, K_{j+2}
            uint32_t pre_p = 0u, pre_v = 0u, pre_k = 0u;

            // Block of K/V tile j (score buffer bc = j & 1): PV(j), then QK(j+2) into the same buffer.
            auto tile_block = [&](auto bc, int j) -> bool {
                constexpr int bsel = decltype(bc)::value;
                const int i = j >> 1;
                const uint32_t tS = tmem_base + (bsel == 0 ? Cfg::kColS0 : Cfg::kColS1);   // P^b overlays it
                const uint32_t tO = tmem_base + (bsel == 0 ? Cfg::kColO0 : Cfg::kColO1);
                const uint32_t vlo = v_lo0 + sv * (Cfg::kVHalfBytes >> 4);
                const uint32_t klo = k_lo0 + sk * (Cfg::kKHalfBytes >> 4);
                const bool more = j + 2 < n_kv;
                if (!pre_v && !duo_wait<false>(smem_addr(&sh.v_full[sv]), ph_v, wctx, kSiteMmaKvFull)) return false;
                if (more && !pre_k && !duo_wait<false>(smem_addr(&sh.k_full[sk]), ph_k, wctx, kSiteMmaKvFull)) return false;
                if (!pre_p && !duo_wait<true>(smem_addr(&sh.p_first[bsel]), i & 1, wctx, kSiteMmaPFull)) return false;
                tc_fence_after_sync();
                // PV k-steps 0..3, then the probe of p_rest under k-steps 4 and 5
                mma2_ts(tO, tS + 0, desc(vlo + 0 * (2048 >> 4)), kIdescPV, i > 0 ? 1u : 0u);
                mma2_ts(tO, tS + 8, desc(vlo + 1 * (2048 >> 4)), kIdescPV, 1u);
                mma2_ts(tO, tS + 16, desc(vlo + 2 * (2048 >> 4)), kIdescPV, 1u);
                mma2_ts(tO, tS + 24, desc(vlo + 3 * (2048 >> 4)), kIdescPV, 1u);
                const uint32_t rest = probe_mma2_ts2(smem_addr(&sh.p_rest[bsel]), i & 1, tO, tS + 32, desc(vlo + 4 * (2048 >> 4)),
                                                     tS + 40, desc(vlo + 5 * (2048 >> 4)), kIdescPV);
                if (!rest && !duo_wait<true>(smem_addr(&sh.p_rest[bsel]), i & 1, wctx, kSiteMmaPFull)) return false;
                tc_fence_after_sync();
                mma2_ts(tO, tS + 48, desc(vlo + 6 * (2048 >> 4)), kIdescPV, 1u);
                mma2_ts(tO, tS + 56, desc(vlo + 7 * (2048 >> 4)), kIdescPV, 1u);
                // stage and phase of V_{j+1} and K_{j+3}
                int sv_n = sv + 1; uint32_t ph_v_n = ph_v; if (sv_n == NV) { sv_n = 0; ph_v_n ^= 1u; }
                int sk_n = sk + 1; uint32_t ph_k_n = ph_k; if (sk_n == NK) { sk_n = 0; ph_k_n ^= 1u; }
                pre_p = pre_v = pre_k = 0u;
                if (more) {
                    mma2_ss(tS, desc(q_lo + qoff(0)), desc(klo + koff(0)), kIdescQK, 0u);
                    mma2_ss(tS, desc(q_lo + qoff(1)), desc(klo + koff(1)), kIdescQK, 1u);
                    mma2_ss(tS, desc(q_lo + qoff(2)), desc(klo + koff(2)), kIdescQK, 1u);
                    mma2_ss(tS, desc(q_lo + qoff(3)), desc(klo + koff(3)), kIdescQK, 1u);
                    // probes: first part of P(j+1) (the other buffer), V_{j+1}, K_{j+3}
                    const bool next_p = j + 1 < n_kv, next_k = j + 3 < n_kv;
                    const uint32_t probed = probe3_mma2_ss3(
                        next_p ? smem_addr(&sh.p_first[bsel ^ 1]) : bar_always, next_p ? (((j + 1) >> 1) & 1) : 0u,
                        next_p ? smem_addr(&sh.v_full[sv_n]) : bar_always, next_p ? ph_v_n : 0u,
                        next_k ? smem_addr(&sh.k_full[sk_n]) : bar_always, next_k ? ph_k_n : 0u,
                        tS, desc(q_lo + qoff(4)), desc(klo + koff(4)), desc(q_lo + qoff(5)), desc(klo + koff(5)),
                        desc(q_lo + qoff(6)), desc(klo + koff(6)), kIdescQK);
                    pre_p = next_p ? (probed & 1u) : 0u;
                    pre_v = next_p ? ((probed >> 1) & 1u) : 0u;
                    pre_k = next_k ? ((probed >> 2) & 1u) : 0u;
#pragma unroll
                    for (int k = 7; k < kKSteps; ++k)
                        mma2_ss(tS, desc(q_lo + qoff(k)), desc(klo + koff(k)), kIdescQK, 1u);
                    tc_commit_2cta(smem_addr(&sh.s_full[bsel]), mapa_shared(smem_addr(&sh.s_full[bsel]), 1u));
                }
                tc_commit_2cta(smem_addr(&sh.v_empty[sv]), mapa_shared(smem_addr(&sh.v_empty[sv]), 1u));
                if (more) tc_commit_2cta(smem_addr(&sh.k_empty[sk]), mapa_shared(smem_addr(&sh.k_empty[sk]), 1u));
                sv = sv_n; ph_v = ph_v_n; sk = sk_n; ph_k = ph_k_n;
                return true;
            };

            for (int j = 0; j < n_kv && ok; j += 2) {
                ok = tile_block(IntC<0>{}, j);
                if (ok && j + 1 < n_kv) ok = tile_block(IntC<1>{}, j + 1);
            }
            if (ok) tc_commit_2cta(smem_addr(&sh.o_final), mapa_shared(smem_addr(&sh.o_final), 1u));
        }
    } else if (warp == 9) {
        // ============================================================ TMA loads: this CTA's Q tile and its halves of K_j, V_j
        setmaxnreg_dec<kPairRegsOther>();
        if (elect_one() && n_kv > 0) {
            const uint32_t bar_q = mapa_shared(smem_addr(&sh.q_full), 0u);
            if (rank == 0) mbar_arrive_expect_tx(smem_addr(&sh.q_full), 2 * Cfg::kQBytes);
#pragma unroll
            for (int cc = 0; cc < Cfg::kQChunks; ++cc)
                tma_load_4d_2cta(sQ + cc * kChunkBytes, &tm_q, bar_q, cc * kChunkCols, i0, hq, b);
            bool ok = true;
            for (int j = 0; j < n_kv && ok; ++j) {
                const int j0 = j * kTileN;
                {
                    const int s = j % NK;
                    ok = duo_wait<false>(smem_addr(&sh.k_empty[s]), ((j / NK) & 1) ^ 1, wctx, kSiteLoadKvEmpty);
                    if (!ok) break;
                    if (rank == 0) mbar_arrive_expect_tx(smem_addr(&sh.k_full[s]), 2 * Cfg::kKHalfBytes);
                    const uint32_t bar = mapa_shared(smem_addr(&sh.k_full[s]), 0u);
#pragma unroll
                    for (int cc = 0; cc < Cfg::kQChunks; ++cc)
                        tma_load_4d_2cta(sK + s * Cfg::kKHalfBytes + cc * Cfg::kKHalfChunkBytes, &tm_k, bar, cc * kChunkCols,
                                         j0 + static_cast<int>(rank) * (kTileN / 2), kvh, b);
                }
                if (!(p.debug_drop_v_load && j == 0)) {
                    const int s = j % NV;
                    ok = duo_wait<false>(smem_addr(&sh.v_empty[s]), ((j / NV) & 1) ^ 1, wctx, kSiteLoadKvEmpty);
                    if (!ok) break;
                    if (rank == 0) mbar_arrive_expect_tx(smem_addr(&sh.v_full[s]), 2 * Cfg::kVHalfBytes);
                    const uint32_t bar = mapa_shared(smem_addr(&sh.v_full[s]), 0u);
                    tma_load_4d_2cta(sV + s * Cfg::kVHalfBytes, &tm_v, bar, static_cast<int>(rank) * kChunkCols, j0, kvh, b);
                }
            }
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
