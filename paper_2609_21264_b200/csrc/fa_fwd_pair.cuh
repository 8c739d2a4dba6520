// Attention forward kernel for sm_100a, head size 128: two 128-row query tiles per CTA, as in
// fa_fwd_pipelined.cuh (read that file first: same tiling, same TMEM map, same arithmetic), with the
// hand-offs of the inner loop cut down to what the dependency chain of a tile needs.
//
// A tile's chain per K/V tile is  S_t(j) visible -> softmax -> P_t(j) -> PV_t(j) -> QK_t(j+1) -> S_t(j+1),
// and with two tiles per SM the period of the loop is the length of that chain.  Measured on B200:
//   * tcgen05.mma 128x128x16 takes 64 cycles, SS or TS, whatever else the SM does, but the tensor pipe
//     queues only about one instruction ahead, so every cycle the issuing thread spends between two
//     MMAs on something else is a cycle the pipe idles;
//   * a probe of an mbarrier whose result is looked at straight away costs the issuing thread well over
//     a hundred cycles while MMAs stream their operands from shared memory; the same probe costs
//     nothing when its result is only read after the next few MMAs have been issued.
// So one thread issues the MMAs of both tiles in a fixed order (tile 0, tile 1, tile 0, ...), and every
// barrier it needs next is probed from inside the block of MMAs before (one asm statement: probe, MMAs,
// then the predicate is read).  Only a probe that failed is followed by a real wait, and then the
// pipe has nothing to do anyway.
//
// There is no correction warpgroup.  The reference maximum moves on a handful of K/V tiles per row (lazy
// rescale, threshold 2^8), so on those tiles the softmax warps multiply their own 32 rows of O_t by
// r = exp(u' - u) in TMEM before they hand P_t over: S_t(j) being visible means PV_t(j-1) is complete,
// and PV_t(j) is not issued before the hand-off.  That removes a role, its barrier, and the rescale
// factors' trip through shared memory from every tile.
//
// P_t is handed over in two parts: keys 0..95 (the PV product starts on them while the last 32
// exponentials are still being computed) and keys 96..127.
//
// Roles (384 threads):
//   warps 0-3, 4-7   softmax of query tile 0 / 1 (one TMEM lane = one query row per thread), rescale of
//                    O_t when needed, final normalisation and stores
//   warp 8           MMA issue (one thread)
//   warp 9           TMA loads of Q_t, K_j, V_j
//   warps 10, 11     idle (they complete the third warpgroup for the register reallocation)
// TMEM: S_0 [0,128) S_1 [128,256) O_0 [256,384) O_1 [384,512); bf16 P_t overlays S_t[0,64).
#pragma once

#include <math.h>

#include "fa_common.cuh"
#include "fa_fwd_pipelined.cuh"
#include "fa_softmax_pass.cuh"
#include "ptx.cuh"

namespace fa {

template <int DQK, int DV>
struct PairCfg {
    static_assert(DQK == 128 && DV == 128, "the pair kernel is written for head size 128");
    static constexpr int kQChunks = DQK / kChunkCols;
    static constexpr int kVChunks = DV / kChunkCols;
    static constexpr int kQBytes = kQChunks * kChunkBytes;    // one query tile
    static constexpr int kKBytes = kQBytes;
    static constexpr int kVBytes = kVChunks * kChunkBytes;
    static constexpr int kKStages = 3;
    static constexpr int kVStages = 2;
    static constexpr int kTileBytes = 2 * kQBytes + kKStages * kKBytes + kVStages * kVBytes;
    static constexpr int kTmemCols = 512;
    static constexpr int kColS0 = 0, kColS1 = 128, kColO0 = 256, kColO1 = 384;
    static constexpr int kThreads = 384;
    static constexpr int kPvFirst = 6;        // k-steps (of 16 keys) of the PV product issued on the first hand-off
};

// Registers per thread after the per-role reallocation (384 threads start with 168 each):
// 256 softmax threads x 216 + 128 other threads x 72 = 64512.
constexpr int kPairRegsSoftmax = 216, kPairRegsOther = 72;
struct PairShared {
    uint64_t q_full[2];
    uint64_t k_full[4], k_empty[4];
    uint64_t v_full[4], v_empty[4];
    uint64_t s_full[2];      // MMA -> softmax: S_t(j) is in TMEM
    uint64_t p_first[2];     // softmax -> MMA: keys 0..95 of P_t(j) written, O_t rescaled if it had to be
    uint64_t p_rest[2];      // softmax -> MMA: all of P_t(j) written
    uint64_t o_final[2];     // MMA -> softmax: last PV of tile t done, O_t is final
    uint64_t o_staged[2];    // softmax warps -> storing thread: the bf16 O_t tile is in shared memory
    uint32_t tmem_base;
    uint32_t abort_flag;
};

template <int DQK, int DV>
constexpr int pair_smem_bytes() {
    return PairCfg<DQK, DV>::kTileBytes + static_cast<int>(sizeof(PairShared));
}

namespace ptx {

// One asm statement: probe up to three mbarriers, issue three SS MMAs (all accumulating), then read
// the probes' predicates.  The probes' latency passes while the MMAs are issued.  Returns a bit per
// probe (1 = that phase is complete).
FA_DEVI uint32_t probe3_mma_ss3(uint32_t bar0, uint32_t par0, uint32_t bar1, uint32_t par1, uint32_t bar2, uint32_t par2,
                                uint32_t d_tmem, uint64_t a0, uint64_t b0, uint64_t a1, uint64_t b1, uint64_t a2, uint64_t b2,
                                uint32_t idesc) {
    uint32_t r;
    asm volatile(
        "{\n"
        ".reg .pred p0, p1, p2, q;\n"
        ".reg .b32 t0, t1, t2;\n"
        "setp.ne.b32 q, 1, 0;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p0, [%1], %2;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p1, [%3], %4;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p2, [%5], %6;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%7], %8, %9, %14, q;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%7], %10, %11, %14, q;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%7], %12, %13, %14, q;\n"
        "selp.u32 t0, 1, 0, p0;\n"
        "selp.u32 t1, 2, 0, p1;\n"
        "selp.u32 t2, 4, 0, p2;\n"
        "or.b32 t0, t0, t1;\n"
        "or.b32 %0, t0, t2;\n"
        "}\n"
        : "=r"(r)
        : "r"(bar0), "r"(par0), "r"(bar1), "r"(par1), "r"(bar2), "r"(par2), "r"(d_tmem), "l"(a0), "l"(b0), "l"(a1),
          "l"(b1), "l"(a2), "l"(b2), "r"(idesc)
        : "memory");
    return r;
}

// Probe one mbarrier, issue two TS MMAs (accumulating), then read the predicate.
FA_DEVI uint32_t probe_mma_ts2(uint32_t bar, uint32_t par, uint32_t d_tmem, uint32_t a0_tmem, uint64_t b0, uint32_t a1_tmem,
                               uint64_t b1, uint32_t idesc) {
    uint32_t r;
    asm volatile(
        "{\n"
        ".reg .pred p0, q;\n"
        "setp.ne.b32 q, 1, 0;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p0, [%1], %2;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%3], [%4], %5, %8, q;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%3], [%6], %7, %8, q;\n"
        "selp.u32 %0, 1, 0, p0;\n"
        "}\n"
        : "=r"(r)
        : "r"(bar), "r"(par), "r"(d_tmem), "r"(a0_tmem), "l"(b0), "r"(a1_tmem), "l"(b1), "r"(idesc)
        : "memory");
    return r;
}

}  // namespace ptx

// kVarlen / kHeadPair as in fa_fwd_pipelined_kernel.
template <int DQK, int DV, bool kVarlen = false, bool kHeadPair = false>
__global__ void __launch_bounds__(384, 1)
fa_fwd_pair_kernel(const __grid_constant__ CUtensorMap tm_q,
                   const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v,
                   const __grid_constant__ CUtensorMap tm_o,
                   const FwdParams p) {
    using Cfg = PairCfg<DQK, DV>;
    using namespace ptx;
    constexpr int NK = Cfg::kKStages;
    constexpr int NV = Cfg::kVStages;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    PairShared& sh = *reinterpret_cast<PairShared*>(smem_raw + Cfg::kTileBytes);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    grid_launch_dependents();
    if constexpr (kVarlen) grid_dependency_wait();

    const uint32_t smem_base = smem_addr(smem_raw);
    if ((smem_base & 1023u) != 0u) {          // uniform over the CTA; nothing has been set up yet
        if constexpr (!kVarlen) grid_dependency_wait();
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

    // Item decode: identical to fa_fwd_pipelined_kernel (L2-sized groups of heads, longest items first).
    const int n_pairs = kHeadPair ? p.n_q_tiles : (p.n_q_tiles + 1) / 2;
    const int n_bh = p.B * p.Hq;
    const int item = static_cast<int>(blockIdx.x) / p.kv_splits;
    const int split = static_cast<int>(blockIdx.x) - item * p.kv_splits;
    const int hpg = kHeadPair ? p.heads_per_group / 2 : p.heads_per_group;
    const int n_units = kHeadPair ? n_bh / 2 : n_bh;
    const int group = item / (n_pairs * hpg);
    const int bh0 = group * hpg;
    const int group_size = (n_units - bh0 < hpg) ? (n_units - bh0) : hpg;
    const int local = item - group * n_pairs * hpg;
    const int pair = n_pairs - 1 - local / group_size;
    const int bh = kHeadPair ? 2 * (bh0 + local % group_size) : bh0 + local % group_size;
    const int hq = bh % p.Hq;
    const int b = bh / p.Hq;
    const int kvh = hq / (p.Hq / p.Hkv);
    const int q_idx = b * p.Hq + hq;
    int Sq = p.Sq, Sk = p.Sk, q_row0 = 0, k_row0 = 0;
    if constexpr (kVarlen) {
        q_row0 = p.cu_q[b];
        k_row0 = p.cu_k[b];
        Sq = p.cu_q[b + 1] - q_row0;
        Sk = p.cu_k[b + 1] - k_row0;
    }
    const int off = Sk - Sq;

    const int i0_0 = (kHeadPair ? pair : 2 * pair) * kTileM, i0_1 = kHeadPair ? i0_0 : i0_0 + kTileM;
    const int j_base = split * p.tiles_per_split;
    auto own_tiles = [&](int i0) -> int {
        if (i0 >= Sq) return 0;
        int n = kv_tiles_for_q_tile(i0, kTileM, Sq, Sk, p.causal) - j_base;
        if (n > p.tiles_per_split) n = p.tiles_per_split;
        return n > 0 ? n : 0;
    };
    const int nkv_0 = own_tiles(i0_0);
    const int nkv_1 = own_tiles(i0_1);
    const int n_max = nkv_0 > nkv_1 ? nkv_0 : nkv_1;
    if (kVarlen && i0_0 >= Sq) return;    // a sequence shorter than the longest one: no rows here

    // ---------------------------------------------------------------- setup
    if (tid == 0) {
        sh.abort_flag = 0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_addr(&sh.q_full[t]), 1);
            mbar_init(smem_addr(&sh.s_full[t]), 1);
            mbar_init(smem_addr(&sh.p_first[t]), 4);      // 4 softmax warps
            mbar_init(smem_addr(&sh.p_rest[t]), 4);
            mbar_init(smem_addr(&sh.o_final[t]), 1);
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
    if constexpr (!kVarlen) grid_dependency_wait();

    const uint32_t tmem_base = sh.tmem_base;
    WaitCtx wctx{&sh.abort_flag, p.status, p.wait_limit_ns};
    const float c = p.scale_log2;

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
        const int i0_t = t == 0 ? i0_0 : i0_1;
        const int hq_t = kHeadPair ? hq + t : hq;
        const int q_idx_t = kHeadPair ? q_idx + t : q_idx;
        const int nkv_t = t == 0 ? nkv_0 : nkv_1;
        const int i_glob = i0_t + row;
        int kmax_row = Sk - 1;
        if (p.causal && i_glob + off < kmax_row) kmax_row = i_glob + off;
        const float tau_raw = kRescaleThresholdLog2 / c;

        float m_ref = -INFINITY;   // reference maximum, raw score units
        float l = 0.f;
        bool ok = true;
        FA_PHASE_DECL();      // phases: 0 wait for S, 5 the pass
        for (int j = 0; j < nkv_t; ++j) {
            ok = __all_sync(0xffffffffu, mbar_wait(bar_s, j & 1, wctx, kSiteSoftmaxSFull));
            if (!ok) break;
            tc_fence_after_sync();
            FA_PHASE(0);
            const int j0 = (j_base + j) * kTileN;
            softmax_pass_128<DV>(tS, tO, c, tau_raw, j0, kmax_row, j == 0, m_ref, l, lane,
                                 [&]() { mbar_arrive(bar_pf); }, [&]() { mbar_arrive(bar_pr); });
            FA_PHASE(5);
        }
        FA_PHASE_STORE(6, nkv_t);
        // epilogue: O = G' / s (bf16), lse = u * scale + ln s   (as in fa_fwd_pipelined_kernel)
        if (ok && i0_t < Sq && p.kv_splits > 1) {
            const size_t prow = (static_cast<size_t>(split) * n_bh + q_idx_t) * p.Sq + i_glob;
            float* po_row = p.o_part + prow * DV;
            bool have = nkv_t > 0;
            if (have) have = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.o_final[t]), 0, wctx, kSiteEpiOFull));
            if (nkv_t == 0 || have) {
                tc_fence_after_sync();
                const float inv_l = (nkv_t > 0 && l > 0.f) ? (1.f / l) : 0.f;
                if (i_glob < Sq)
                    p.lse_part[prow] = (nkv_t > 0 && l > 0.f) ? (m_ref * c * 0.6931471805599453f + logf(l)) : -INFINITY;
#pragma unroll 1
                for (int cc = 0; cc < DV / 32; ++cc) {
                    uint32_t r[32];
                    if (nkv_t > 0) {
                        tmem_ld_x32(tO + cc * 32, r);
                        tc_wait_ld();
                    }
                    if (i_glob < Sq) {
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            float4 f;
                            f.x = (nkv_t > 0) ? __uint_as_float(r[4 * v]) * inv_l : 0.f;
                            f.y = (nkv_t > 0) ? __uint_as_float(r[4 * v + 1]) * inv_l : 0.f;
                            f.z = (nkv_t > 0) ? __uint_as_float(r[4 * v + 2]) * inv_l : 0.f;
                            f.w = (nkv_t > 0) ? __uint_as_float(r[4 * v + 3]) * inv_l : 0.f;
                            reinterpret_cast<float4*>(po_row + cc * 32)[v] = f;
                        }
                    }
                }
            }
        } else if (ok && i0_t < Sq) {
            const size_t lse_row0 = kVarlen ? static_cast<size_t>(hq_t) * p.total_q + q_row0
                                           : static_cast<size_t>(q_idx_t) * p.Sq;
            const long long o_base = (kVarlen ? q_row0 * p.o_stride_s : b * p.o_stride_b) + hq_t * p.o_stride_h;
            __nv_bfloat16* o_row = p.O + (o_base + static_cast<long long>(i_glob) * p.o_stride_s);
            if (nkv_t == 0) {         // no key visible to any row of this tile
                if (i_glob < Sq) {
                    const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int v = 0; v < DV / 8; ++v) reinterpret_cast<uint4*>(o_row)[v] = z;
                    if (p.lse) p.lse[lse_row0 + i_glob] = -INFINITY;
                }
            } else if (__all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.o_final[t]), 0, wctx, kSiteEpiOFull))) {
                tc_fence_after_sync();
                const float inv_l = (l > 0.f) ? (1.f / l) : 0.f;
                if (p.lse && i_glob < Sq) {
                    p.lse[lse_row0 + i_glob] =
                        (l > 0.f) ? (m_ref * c * 0.6931471805599453f + logf(l)) : -INFINITY;
                }
                const bool box_store = !kVarlen || (i0_t + kTileM <= Sq);
                {
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
                }
                if (box_store) {
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_addr(&sh.o_staged[t]));
                    if ((warp & 3) == 0 && lane == 0 &&
                        mbar_wait(smem_addr(&sh.o_staged[t]), 0, wctx, kSiteEpiStaged)) {
#pragma unroll
                        for (int ch = 0; ch < DV / kChunkCols; ++ch)
                            tma_store_4d(&tm_o, sQ + t * Cfg::kQBytes + ch * kChunkBytes, ch * kChunkCols,
                                         q_row0 + i0_t, hq_t, kVarlen ? 0 : b);
                        tma_store_commit();
                        tma_store_wait_read_all();     // the CTA's shared memory outlives the reads
                    }
                } else {
                    __syncwarp();
                    store_staged_rows<DV>(sQ + t * Cfg::kQBytes, (warp & 3) * 32, Sq - i0_t,
                                          o_row - static_cast<long long>(row) * p.o_stride_s, p.o_stride_s, lane);
                }
            }
        }
    } else if (warp == 8) {
        // ============================================================ MMA issue, one thread for both tiles
        setmaxnreg_dec<kPairRegsOther>();
        // elect.sync, not lane == 0: only then are the descriptors kept in uniform registers (see the top of the file)
        if (elect_one() && n_max > 0) {
            constexpr uint32_t kIdescQK = make_idesc_bf16_f32(kTileM, kTileN, false, false);
            constexpr uint32_t kIdescPV = make_idesc_bf16_f32(kTileM, DV, false, true);
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // sbo, version, swizzle
            const uint32_t q_lo0 = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t v_lo0 = ((sV & 0x3FFFFu) >> 4) | ((static_cast<uint32_t>(kChunkBytes) >> 4) << 16);
            auto desc = [](uint32_t lo) -> uint64_t {
                return (static_cast<uint64_t>(kDescHi) << 32) | lo;
            };
            auto koff = [](int k) -> uint32_t { return static_cast<uint32_t>(((k / 4) * kChunkBytes + (k % 4) * 32) >> 4); };
            // a barrier whose phase 0 completed long ago and which never moves again: filler for unused probe slots
            const uint32_t bar_always = smem_addr(&sh.q_full[nkv_0 > 0 ? 0 : 1]);

            bool ok = mbar_wait(smem_addr(&sh.k_full[0]), 0, wctx, kSiteMmaKvFull);
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (ok && (t == 0 ? nkv_0 : nkv_1) > 0) {
                    ok = mbar_wait(smem_addr(&sh.q_full[t]), 0, wctx, kSiteMmaQFull);
                    if (ok) {
                        tc_fence_after_sync();
                        const uint32_t tS = tmem_base + (t == 0 ? Cfg::kColS0 : Cfg::kColS1);
                        const uint32_t q_lo = q_lo0 + t * (Cfg::kQBytes >> 4);
#pragma unroll
                        for (int k = 0; k < DQK / 16; ++k)
                            mma_ss(tS, desc(q_lo + koff(k)), desc(k_lo0 + koff(k)), kIdescQK, k > 0 ? 1u : 0u);
                        tc_commit(smem_addr(&sh.s_full[t]));
                    }
                }
            }
            if (ok) tc_commit(smem_addr(&sh.k_empty[0]));
            int sv = 0, sk = (NK > 1) ? 1 : 0;       // stage of V_j and of K_{j+1}
            uint32_t ph_v = 0, ph_k = (NK > 1) ? 0u : 1u;
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
                const uint32_t vlo = v_lo0 + sv * (Cfg::kVBytes >> 4);
                const uint32_t klo = k_lo0 + sk * (Cfg::kKBytes >> 4);
                FA_PHASE(0);
                if (!pre_first && !mbar_wait(smem_addr(&sh.p_first[t]), j & 1, wctx, kSiteMmaPFull)) return false;
                FA_PHASE(1);
                tc_fence_after_sync();
                // PV k-steps 0..3, then the probe of p_rest under k-steps 4 and 5
                mma_ts(tO, tS + 0, desc(vlo + 0 * (2048 >> 4)), kIdescPV, j > 0 ? 1u : 0u);
                mma_ts(tO, tS + 8, desc(vlo + 1 * (2048 >> 4)), kIdescPV, 1u);
                mma_ts(tO, tS + 16, desc(vlo + 2 * (2048 >> 4)), kIdescPV, 1u);
                mma_ts(tO, tS + 24, desc(vlo + 3 * (2048 >> 4)), kIdescPV, 1u);
                const uint32_t rest = probe_mma_ts2(smem_addr(&sh.p_rest[t]), j & 1, tO, tS + 32, desc(vlo + 4 * (2048 >> 4)),
                                                    tS + 40, desc(vlo + 5 * (2048 >> 4)), kIdescPV);
                FA_PHASE(2);
                if (!rest && !mbar_wait(smem_addr(&sh.p_rest[t]), j & 1, wctx, kSiteMmaPFull)) return false;
                FA_PHASE(3);
                tc_fence_after_sync();
                mma_ts(tO, tS + 48, desc(vlo + 6 * (2048 >> 4)), kIdescPV, 1u);
                mma_ts(tO, tS + 56, desc(vlo + 7 * (2048 >> 4)), kIdescPV, 1u);
                if (j + 1 < nkv_t) {
                    mma_ss(tS, desc(q_lo + koff(0)), desc(klo + koff(0)), kIdescQK, 0u);
                    mma_ss(tS, desc(q_lo + koff(1)), desc(klo + koff(1)), kIdescQK, 1u);
                    mma_ss(tS, desc(q_lo + koff(2)), desc(klo + koff(2)), kIdescQK, 1u);
                    mma_ss(tS, desc(q_lo + koff(3)), desc(klo + koff(3)), kIdescQK, 1u);
                    probed = probe3_mma_ss3(b0, par0, b1, par1, b2, par2, tS, desc(q_lo + koff(4)), desc(klo + koff(4)),
                                            desc(q_lo + koff(5)), desc(klo + koff(5)), desc(q_lo + koff(6)), desc(klo + koff(6)),
                                            kIdescQK);
                    mma_ss(tS, desc(q_lo + koff(7)), desc(klo + koff(7)), kIdescQK, 1u);
                    tc_commit(smem_addr(&sh.s_full[t]));
                } else {
                    tc_commit(smem_addr(&sh.o_final[t]));
                }
                FA_PHASE(4);
                return true;
            };

            for (int j = 0; j < n_max && ok; ++j) {
                FA_PHASE(0);
                if (!pre_v) ok = mbar_wait(smem_addr(&sh.v_full[sv]), ph_v, wctx, kSiteMmaKvFull);
                if (ok && j + 1 < n_max && !pre_k) ok = mbar_wait(smem_addr(&sh.k_full[sk]), ph_k, wctx, kSiteMmaKvFull);
                if (!ok) break;
                FA_PHASE(5);
#if defined(FA_TRACE) && defined(FA_TRACE_PHASES)
                ph_acc[6] += (pre_v ? 0u : 1u) + (pre_k ? 0u : 1000u) + (pre_p0 ? 0u : 1000000u);
#endif
                uint32_t probed;
                // block of tile 0; probes: first part of P_1(j)
                ok = tile_block(IntC<0>{}, j, nkv_0, pre_p0, (j < nkv_1) ? smem_addr(&sh.p_first[1]) : bar_always,
                                (j < nkv_1) ? (j & 1) : 0u, bar_always, 0u, bar_always, 0u, probed);
                if (!ok) break;
                pre_p1 = (j < nkv_1) ? (probed & 1u) : 0u;
                // stage and phase of V_{j+1} and K_{j+2}
                int sv_n = sv + 1; uint32_t ph_v_n = ph_v; if (sv_n == NV) { sv_n = 0; ph_v_n ^= 1u; }
                int sk_n = sk + 1; uint32_t ph_k_n = ph_k; if (sk_n == NK) { sk_n = 0; ph_k_n ^= 1u; }
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
                tc_commit(smem_addr(&sh.v_empty[sv]));
                if (j + 1 < n_max) tc_commit(smem_addr(&sh.k_empty[sk]));
                sv = sv_n; ph_v = ph_v_n; sk = sk_n; ph_k = ph_k_n;
            }
            FA_PHASE_STORE(7, n_max);
        }
    } else if (warp == 9) {
        // ============================================================ TMA loads
        setmaxnreg_dec<kPairRegsOther>();
        if (elect_one() && n_max > 0) {
            auto load_q = [&](int t) {
                if ((t == 0 ? nkv_0 : nkv_1) == 0) return;
                const uint32_t bar = smem_addr(&sh.q_full[t]);
                mbar_arrive_expect_tx(bar, Cfg::kQBytes);
#pragma unroll
                for (int cc = 0; cc < Cfg::kQChunks; ++cc)
                    tma_load_4d(sQ + t * Cfg::kQBytes + cc * kChunkBytes, &tm_q, bar, cc * kChunkCols,
                                q_row0 + (t == 0 ? i0_0 : i0_1), kHeadPair ? hq + t : hq, kVarlen ? 0 : b);
            };
            load_q(0);
            bool ok = true;
            for (int j = 0; j < n_max && ok; ++j) {
                const int j0 = (j_base + j) * kTileN;
                {
                    const int s = j % NK;
                    ok = mbar_wait(smem_addr(&sh.k_empty[s]), ((j / NK) & 1) ^ 1, wctx, kSiteLoadKvEmpty);
                    if (!ok) break;
                    const uint32_t bar = smem_addr(&sh.k_full[s]);
                    mbar_arrive_expect_tx(bar, Cfg::kKBytes);
#pragma unroll
                    for (int cc = 0; cc < Cfg::kQChunks; ++cc)
                        tma_load_4d(sK + s * Cfg::kKBytes + cc * kChunkBytes, &tm_k, bar, cc * kChunkCols,
                                    k_row0 + j0, kvh, kVarlen ? 0 : b);
                    if (j == 0) load_q(1);
                }
                if (!(p.debug_drop_v_load && j == 0)) {
                    const int s = j % NV;
                    ok = mbar_wait(smem_addr(&sh.v_empty[s]), ((j / NV) & 1) ^ 1, wctx, kSiteLoadKvEmpty);
                    if (!ok) break;
                    const uint32_t bar = smem_addr(&sh.v_full[s]);
                    mbar_arrive_expect_tx(bar, Cfg::kVBytes);
#pragma unroll
                    for (int cc = 0; cc < Cfg::kVChunks; ++cc)
                        tma_load_4d(sV + s * Cfg::kVBytes + cc * kChunkBytes, &tm_v, bar, cc * kChunkCols,
                                    k_row0 + j0, kvh, kVarlen ? 0 : b);
                }
            }
        }
    } else {
        setmaxnreg_dec<kPairRegsOther>();     // idle warps of the third warpgroup
    }

    // ---------------------------------------------------------------- teardown (all warps)
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem_base, Cfg::kTmemCols);
}

}  // namespace fa
