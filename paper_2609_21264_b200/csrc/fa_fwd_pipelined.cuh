// Pipelined, warp-specialised attention forward kernel for sm_100a.
//
// One CTA owns two adjacent 128-row query tiles of one (batch, query head) and
// walks the K/V tiles they can see.  Roles:
//   warps 0-3   softmax of query tile 0 (one TMEM lane = one query row per thread), then its
//               final normalisation and stores
//   warps 4-7   softmax of query tile 1
//   warps 8-11  correction: rescale of the O accumulators when a reference maximum moved
//   warps 12,13 MMA issue (one thread each, one per query tile): S_t = Q_t K_j^T and
//               O_t += P_t V_j with tcgen05
//   warp  14    TMA loads of Q_t, K_j, V_j into mbarrier-guarded shared-memory rings
//   warp  15    idle (it keeps the fourth warpgroup complete)
// While one softmax warpgroup works on S_t(j), the tensor core runs the MMAs of
// the other tile, so the exponentials overlap the contractions.
//
// The recurrence is Algorithm 1 with fp32 state: running row maximum u, running
// row sum s, unnormalised accumulator G' in TMEM, P rounded to bf16 before the
// second contraction, one division at the end (Section 2.1).  Two deviations in
// evaluation order, neither changing the result beyond rounding:
//   * the scale 1/sqrt(dk) is folded into the exponent (exp2((g - u) * scale *
//     log2 e)) instead of being applied to Q, so Q is never re-rounded;
//   * the reference maximum u is only advanced when the row maximum grew by more
//     than 2^8 in the exponent, so the rescale r = exp(u' - u) of G' is skipped
//     on most tiles; G' and s are always expressed against the same u, and the
//     final G'/s and lse = u + ln s are unchanged.
// TMEM: S_0 [0,128) S_1 [128,256) O_0 [256,256+dv) O_1 [384,384+dv); bf16 P_t
// overlays the first 64 columns of S_t.
#pragma once

#include <math.h>

#include "fa_common.cuh"
#include "ptx.cuh"

namespace fa {

template <int DQK, int DV>
struct PipeCfg {
    static constexpr int kQChunks = DQK / kChunkCols;
    static constexpr int kVChunks = DV / kChunkCols;
    static constexpr int kQBytes = kQChunks * kChunkBytes;    // one query tile
    static constexpr int kKBytes = kQBytes;
    static constexpr int kVBytes = kVChunks * kChunkBytes;
    static constexpr int kKStages = (DQK == 192) ? 2 : (DQK == 128 ? 3 : 4);
    static constexpr int kVStages = (DQK == 192) ? 1 : (DQK == 128 ? 2 : 4);
    static constexpr int kTileBytes = 2 * kQBytes + kKStages * kKBytes + kVStages * kVBytes;
    static constexpr int kTmemCols = 512;
    static constexpr int kColS0 = 0, kColS1 = 128, kColO0 = 256, kColO1 = 384;
    // At head size 64 an O accumulator takes 64 columns and the 64 behind it hold P_t, so that
    // P_t(j) does not overlay S_t: the score MMA of K/V tile j+1 is then issued as soon as the softmax
    // warps hold S_t(j) in registers, and a tile's chain is softmax -> softmax instead of
    // softmax -> PV -> QK.  (At 128 the 512 columns are taken by 2 x (S + O) and P_t overlays S_t.)
    static constexpr bool kSeparateP = (DV == 64);
    static constexpr int kColP0 = kSeparateP ? kColO0 + 64 : kColS0, kColP1 = kSeparateP ? kColO1 + 64 : kColS1;
    static constexpr int kThreads = 512;
};

template <int V>
struct IntC { static constexpr int value = V; };

constexpr float kRescaleThresholdLog2 = 8.0f;
// Registers per thread after the per-role reallocation (512 threads start with 128 each):
// 256 softmax threads x 192 + 128 correction threads x 64 + 128 other threads x 64 = 65536.
constexpr int kRegsSoftmax = 192, kRegsCorrection = 64, kRegsOther = 64;

struct PipeShared {
    uint64_t q_full[2];
    uint64_t k_full[4], k_empty[4];
    uint64_t v_full[4], v_empty[4];
    uint64_t s_full[2];      // MMA -> softmax: S_t(j) is in TMEM
    uint64_t p_half[2];      // softmax + correction -> MMA: keys 0..63 of P_t(j) written, O_t rescaled
    uint64_t p_full[2];      // softmax -> MMA: all of P_t(j) written
    uint64_t scale_full[2];  // softmax -> correction: alpha of iteration j published
    uint64_t o_final[2];     // MMA -> softmax: last PV of tile t done, O_t is final
    uint64_t turn[2];        // MMA thread 1-t -> MMA thread t: your turn to issue
    uint64_t o_staged[2];    // softmax warps -> storing thread: the bf16 O_t tile is in shared memory
    uint64_t pv_done[2];     // MMA -> softmax, correction (separate P only): PV of iteration j complete, P_t and O_t may be written
    uint64_t s_read[2];      // softmax -> MMA (separate P only): S_t(j) is in registers, the next score block may be issued
    float alpha[2][2][kTileM];   // [tile][j & 1][row]
    uint32_t tmem_base;
    uint32_t abort_flag;
};

template <int DQK, int DV>
constexpr int pipe_smem_bytes() {
    return PipeCfg<DQK, DV>::kTileBytes + static_cast<int>(sizeof(PipeShared));
}

// kVarlen = packed variable-length batch (per-sequence offsets and lengths read from p.cu_q/p.cu_k);
// a template parameter so that the fixed-length instantiation carries none of its scalars.
// kHeadPair = the CTA's two query tiles are the SAME query tile of two adjacent query heads that share
// a K/V head (grouped-query attention with an even group size) instead of two adjacent query tiles
// of one head.  With a causal mask both tiles then see the same number of K/V tiles, so neither
// runs a last round alone, and the items come in lengths 1, 2, 3, ... instead of 2, 4, 6, ...
template <int DQK, int DV, bool kVarlen = false, bool kHeadPair = false>
__global__ void __launch_bounds__(512, 1)
fa_fwd_pipelined_kernel(const __grid_constant__ CUtensorMap tm_q,
                        const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v,
                        const __grid_constant__ CUtensorMap tm_o,
                        const FwdParams p) {
    using Cfg = PipeCfg<DQK, DV>;
    using namespace ptx;
    constexpr int NK = Cfg::kKStages;
    constexpr int NV = Cfg::kVStages;

    // All shared memory is dynamic: the swizzled tiles first (they need a 1024-byte aligned
    // base), the barriers and hand-off buffers behind them.
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    PipeShared& sh = *reinterpret_cast<PipeShared*>(smem_raw + Cfg::kTileBytes);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    // The launch after this one may be scheduled while this grid drains; the inputs of this
    // launch are not touched before the launch before it has completed.  Packed batches read their
    // offsets right away, so they wait here; otherwise the wait comes after the CTA's set-up.
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
#ifdef FA_TRACE
    if (tid == 0 && p.trace) {      // per-CTA record: SM id, start, end, rounds (after the role stamps)
        unsigned long long g; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(g));
        unsigned smid; asm volatile("mov.u32 %0, %smid;" : "=r"(smid));
        long long* rec = p.trace + kTraceRoles * kTraceIters * kTraceEvents + 4ll * blockIdx.x;
        rec[0] = smid; rec[1] = static_cast<long long>(g);
    }
#endif
    const uint32_t sQ = smem_base;                               // two tiles
    const uint32_t sK = sQ + 2 * Cfg::kQBytes;                   // NK stages
    const uint32_t sV = sK + NK * Cfg::kKBytes;                  // NV stages

    // 1-D grid.  The (batch, head) instances are cut into groups whose K/V fit in L2 together;
    // groups run one after the other, and inside a group the CTAs are in longest-processing-time
    // order: every head's last (with a causal mask: heaviest) pair of query tiles first, then the
    // pair before it, and so on.  Consecutive CTAs are consecutive query heads (shared K/V heads).
    // (kHeadPair: an item is one query tile of a pair of heads; bh then counts pairs of heads)
    const int n_pairs = kHeadPair ? p.n_q_tiles : (p.n_q_tiles + 1) / 2;
    const int n_bh = p.B * p.Hq;
    // With split-KV (the spatial decomposition of Algorithm 2) the C CTAs that share an item's
    // query tiles and take disjoint ranges of its K/V tiles are adjacent in the grid.
    const int item = static_cast<int>(blockIdx.x) / p.kv_splits;
    const int split = static_cast<int>(blockIdx.x) - item * p.kv_splits;
    const int hpg = kHeadPair ? p.heads_per_group / 2 : p.heads_per_group;     // (pairs of) heads per group
    const int n_units = kHeadPair ? n_bh / 2 : n_bh;
    const int group = item / (n_pairs * hpg);
    const int bh0 = group * hpg;
    const int group_size = (n_units - bh0 < hpg) ? (n_units - bh0) : hpg;
    const int local = item - group * n_pairs * hpg;
    const int pair = n_pairs - 1 - local / group_size;
    const int bh = kHeadPair ? 2 * (bh0 + local % group_size) : bh0 + local % group_size;   // first head of the item
    const int hq = bh % p.Hq;
    const int b = bh / p.Hq;
    const int kvh = hq / (p.Hq / p.Hkv);
    const int q_idx = b * p.Hq + hq;
    // Problem of this CTA: Sq x Sk, its Q rows starting at q_row0 and K/V rows at k_row0 of the
    // tensors the maps describe (packed variable-length tensors are one batch slice).
    int Sq = p.Sq, Sk = p.Sk, q_row0 = 0, k_row0 = 0;
    if constexpr (kVarlen) {
        q_row0 = p.cu_q[b];
        k_row0 = p.cu_k[b];
        Sq = p.cu_q[b + 1] - q_row0;
        Sk = p.cu_k[b + 1] - k_row0;
    }
    const int off = Sk - Sq;

    // per-tile scalars (no arrays: a runtime-indexed array would live in local memory)
    const int i0_0 = (kHeadPair ? pair : 2 * pair) * kTileM, i0_1 = kHeadPair ? i0_0 : i0_0 + kTileM;
    // K/V tiles [j_base, j_base + nkv_t) of tile t belong to this CTA (all visible ones without split-KV)
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
    if (kVarlen && i0_0 >= Sq) return;    // a sequence shorter than the longest one: no rows here (whole CTA, before any set-up)

    // ---------------------------------------------------------------- setup
    if (tid == 0) {
        sh.abort_flag = 0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_addr(&sh.q_full[t]), 1);
            mbar_init(smem_addr(&sh.s_full[t]), 1);
            mbar_init(smem_addr(&sh.p_half[t]), 8);       // 4 softmax warps + 4 correction warps
            mbar_init(smem_addr(&sh.p_full[t]), 4);       // 4 softmax warps
            mbar_init(smem_addr(&sh.scale_full[t]), 4);
            mbar_init(smem_addr(&sh.o_final[t]), 1);
            mbar_init(smem_addr(&sh.turn[t]), 1);
            mbar_init(smem_addr(&sh.o_staged[t]), 4);     // 4 softmax warps
            mbar_init(smem_addr(&sh.pv_done[t]), 1);
            mbar_init(smem_addr(&sh.s_read[t]), 4);       // 4 softmax warps
        }
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            mbar_init(smem_addr(&sh.k_full[s]), 1);
            mbar_init(smem_addr(&sh.k_empty[s]), 2);      // one arrival per MMA-issuing thread
            mbar_init(smem_addr(&sh.v_full[s]), 1);
            mbar_init(smem_addr(&sh.v_empty[s]), 2);
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
    if constexpr (!kVarlen) grid_dependency_wait();

    const uint32_t tmem_base = sh.tmem_base;
    WaitCtx wctx{&sh.abort_flag, p.status, p.wait_limit_ns};
    const float c = p.scale_log2;

    if (warp < 8) {
        // ============================================================ softmax of tile t
        setmaxnreg_inc<kRegsSoftmax>();
        const int t = warp >> 2;
        const int row = tid & (kTileM - 1);
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + (t == 0 ? Cfg::kColS0 : Cfg::kColS1) + lane_sel;
        const uint32_t tP = tmem_base + (t == 0 ? Cfg::kColP0 : Cfg::kColP1) + lane_sel;
        const uint32_t bar_s = smem_addr(&sh.s_full[t]);
        const uint32_t bar_p = smem_addr(&sh.p_full[t]);
        const uint32_t bar_ph = smem_addr(&sh.p_half[t]);
        const uint32_t bar_scale = smem_addr(&sh.scale_full[t]);
        const int i0_t = t == 0 ? i0_0 : i0_1;
        const int hq_t = kHeadPair ? hq + t : hq;          // query head of this tile
        const int q_idx_t = kHeadPair ? q_idx + t : q_idx;
        const int nkv_t = t == 0 ? nkv_0 : nkv_1;
        const int i_glob = i0_t + row;
        int kmax_row = Sk - 1;
        if (p.causal && i_glob + off < kmax_row) kmax_row = i_glob + off;
        const float tau_raw = kRescaleThresholdLog2 / c;

        float m_ref = -INFINITY;   // reference maximum, raw score units
        float l = 0.f;
        bool ok = true;
        for (int j = 0; j < nkv_t; ++j) {
            ok = __all_sync(0xffffffffu, mbar_wait(bar_s, j & 1, wctx, kSiteSoftmaxSFull));
            if (!ok) break;
            tc_fence_after_sync();
            if (lane == 0 && ((warp & 3) == 0 || (warp & 3) == 2)) FA_TRACE_STAMP(t + ((warp & 3) == 2 ? 4 : 0), j, 0);
            const int j0 = (j_base + j) * kTileN;
            const bool need_mask = (j0 + kTileN - 1 > kmax_row);

            const float2 c2 = make_float2(c, c);
            float2 nmc2;
            float2 sum_a = make_float2(0.f, 0.f), sum_b = make_float2(0.f, 0.f);
            float alpha = 1.f;
            uint32_t s[kTileN];
            // Exponentials in place against the reference maximum (packed FMA for the argument).
            auto exp_chunk = [&](int q) {
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[q * 32 + e]),
                                                            __uint_as_float(s[q * 32 + e + 1])), c2, nmc2);
                    s[q * 32 + e] = __float_as_uint(exp2_approx(x.x));
                    s[q * 32 + e + 1] = __float_as_uint(exp2_approx(x.y));
                }
            };
            // Row sum, bf16 conversion and store of one chunk of P (over the first half of S).
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
            // The exponentials do not wait for the row maximum: they start against the reference
            // maximum carried over from earlier tiles while the maximum of this tile is reduced on
            // the ALU pipe.  Only if some row of the warp grew past the threshold (always on the
            // first tile, rarely afterwards) is the reference advanced and the pass repeated; no
            // P has been stored yet at that point, so S is still intact in TMEM.
#pragma unroll 1
            for (;;) {
                tmem_ld_x32(tS + 0, s + 0);
                tmem_ld_x32(tS + 32, s + 32);
                tmem_ld_x32(tS + 64, s + 64);
                tmem_ld_x32(tS + 96, s + 96);
                tc_wait_ld();
                if (lane == 0 && ((warp & 3) == 0 || (warp & 3) == 2)) FA_TRACE_STAMP(t + ((warp & 3) == 2 ? 4 : 0), j, 1);
                if (need_mask) {
#pragma unroll
                    for (int e = 0; e < kTileN; ++e)
                        if (j0 + e > kmax_row) s[e] = 0xff800000u;   // -inf
                }
                const float mc = (m_ref == -INFINITY) ? 0.f : m_ref * c;
                nmc2 = make_float2(-mc, -mc);
                float a[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) a[q] = -INFINITY;
#pragma unroll
                for (int e = 0; e < kTileN; e += 16) {
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        a[q] = fmax3(a[q], __uint_as_float(s[e + 2 * q]), __uint_as_float(s[e + 2 * q + 1]));
                }
                exp_chunk(0);
                float mx = fmaxf(fmax3(a[0], a[1], a[2]), fmax3(a[3], a[4], a[5]));
                mx = fmax3(mx, a[6], a[7]);
                const bool grow = mx > m_ref + tau_raw;
                if (!__any_sync(0xffffffffu, grow)) break;
                if (grow) {
                    alpha = exp2_approx((m_ref - mx) * c);    // r = exp(u' - u); 0 on the first tile
                    m_ref = mx;
                }
            }
            sh.alpha[t][j & 1][row] = alpha;
            if constexpr (Cfg::kSeparateP) {
                // S_t(j) is in registers: the next score block may overwrite it.
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_addr(&sh.s_read[t]));
                // P_t(j-1) is still being read by its PV product unless that has completed.  The wait
                // comes before the rescale factor is published, not just before the first store of
                // P_t(j): the softmax no longer follows the PV product on the tensor pipe, and without it
                // scale_full could run two phases ahead of the correction warps.
                if (j > 0) {
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.pv_done[t]), (j - 1) & 1, wctx, kSiteSoftmaxPFree));
                    if (!ok) break;
                    tc_fence_after_sync();
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_scale);
            if (lane == 0 && ((warp & 3) == 0 || (warp & 3) == 2)) FA_TRACE_STAMP(t + ((warp & 3) == 2 ? 4 : 0), j, 2);

            exp_chunk(1);
            emit_chunk(0);
            exp_chunk(2);
            emit_chunk(1);
            exp_chunk(3);
            // first half of P (keys 0..63) is stored: the MMA thread may start O += P V on it
            tc_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_ph);
            emit_chunk(2);
            emit_chunk(3);
            l = l * alpha + ((sum_a.x + sum_a.y) + (sum_b.x + sum_b.y));
            if (lane == 0 && ((warp & 3) == 0 || (warp & 3) == 2)) FA_TRACE_STAMP(t + ((warp & 3) == 2 ? 4 : 0), j, 3);
            tc_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_p);
            if (lane == 0 && ((warp & 3) == 0 || (warp & 3) == 2)) FA_TRACE_STAMP(t + ((warp & 3) == 2 ? 4 : 0), j, 4);
        }
        // epilogue: O = G' / s (bf16), lse = u * scale + ln s
        if (ok && i0_t < Sq && p.kv_splits > 1) {
            // split-KV: this CTA's partial (G'_c / s_c in fp32, and u_c + ln s_c) goes to scratch;
            // the combine kernel merges the C partials of a row (Algorithm 2's reduction).
            const size_t prow = (static_cast<size_t>(split) * n_bh + q_idx_t) * p.Sq + i_glob;
            float* po_row = p.o_part + prow * DV;
            bool have = nkv_t > 0;
            if (have) have = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.o_final[t]), 0, wctx, kSiteEpiOFull));
            if (nkv_t == 0 || have) {
                tc_fence_after_sync();
                const float inv_l = (nkv_t > 0 && l > 0.f) ? (1.f / l) : 0.f;
                if (i_glob < Sq)
                    p.lse_part[prow] = (nkv_t > 0 && l > 0.f) ? (m_ref * c * 0.6931471805599453f + logf(l)) : -INFINITY;
                const uint32_t tO = tmem_base + (t == 0 ? Cfg::kColO0 : Cfg::kColO1) + lane_sel;
#pragma unroll 1
                for (int cc = 0; cc < DV / 32; ++cc) {
                    uint32_t r[32];
                    if (nkv_t > 0) {            // uniform over the CTA's tile: warp-collective load is safe
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
            // fixed lengths: lse [B, Hq, Sq]; packed batches: lse [Hq, total_q], O rows q_row0 onwards
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
                const uint32_t tO = tmem_base + (t == 0 ? Cfg::kColO0 : Cfg::kColO1) + lane_sel;
                // A packed batch's last tile of a sequence is followed by the next sequence's rows,
                // which a box store would overwrite: such tiles take the row-by-row path.
                const bool box_store = !kVarlen || (i0_t + kTileM <= Sq);
                {
                    // The tile goes through shared memory (the Q tile's space: its last reader, the
                    // final score MMA, is complete once o_final has fired) in the swizzled layout of
                    // a TMA box, and one thread stores it; rows past Sq are clipped by the TMA unit.
                    // Row-by-row global stores from 128 threads cost one LSU pass per 16 bytes.
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
                    // every warp copies the 32 rows it staged itself, whole rows per instruction
                    __syncwarp();
                    store_staged_rows<DV>(sQ + t * Cfg::kQBytes, (warp & 3) * 32, Sq - i0_t,
                                          o_row - static_cast<long long>(row) * p.o_stride_s, p.o_stride_s, lane);
                }
            }
        }
    } else if (warp < 12) {
        // ============================================================ correction of the O accumulators
        setmaxnreg_dec<kRegsCorrection>();
        const int row = tid & (kTileM - 1);
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        bool ok = true;
        for (int j = 0; j < n_max && ok; ++j) {
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (j >= (t == 0 ? nkv_0 : nkv_1) || !ok) continue;
                ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.scale_full[t]), j & 1, wctx,
                                                       kSiteCorrScale));
                if (!ok) break;
                const float alpha = sh.alpha[t][j & 1][row];
                if constexpr (Cfg::kSeparateP) {
                    // the score block of iteration j no longer follows the PV product of j-1 on the tensor pipe
                    if (j > 0) {
                        ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.pv_done[t]), (j - 1) & 1, wctx, kSiteCorrPvDone));
                        if (!ok) break;
                    }
                }
                if (lane == 0 && (warp & 3) == 0) FA_TRACE_STAMP(3, j, t * 4 + 0);
                if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                    tc_fence_after_sync();
                    const uint32_t tO = tmem_base + (t == 0 ? Cfg::kColO0 : Cfg::kColO1) + lane_sel;
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
                if (lane == 0) mbar_arrive(smem_addr(&sh.p_half[t]));
                if (lane == 0 && (warp & 3) == 0) FA_TRACE_STAMP(3, j, t * 4 + 1);
            }
        }
    } else if (warp == 12 || warp == 13) {
        // ============================================================ MMA issue for tile t = warp - 12
        // One issuing thread per query tile: tcgen05.mma issue blocks while the tensor pipe is
        // busy, so a single thread serving both tiles would serialise their waits behind each
        // other's MMAs.  The two threads touch disjoint TMEM (S_t, O_t) and share the K/V stages,
        // whose "empty" barriers therefore count two arrivals.
        setmaxnreg_dec<kRegsOther>();
        if (elect_one() && n_max > 0) {
            const int t = warp - 12;
            const int nkv_t = (t == 0) ? nkv_0 : nkv_1;
            constexpr uint32_t kIdescQK = make_idesc_bf16_f32(kTileM, kTileN, false, false);
            constexpr uint32_t kIdescPV = make_idesc_bf16_f32(kTileM, DV, false, true);
            // Descriptor words are built once.  Per MMA only the 14-bit start-address field of the
            // low word moves (shared-memory addresses stay below 2^18, so no carry leaves it).
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // sbo, version, swizzle
            const uint32_t q_lo = (((sQ + t * Cfg::kQBytes) & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t v_lo0 = ((sV & 0x3FFFFu) >> 4) | ((static_cast<uint32_t>(kChunkBytes) >> 4) << 16);
            const uint32_t tS = tmem_base + (t == 0 ? Cfg::kColS0 : Cfg::kColS1);   // P_t overlays it unless kSeparateP
            const uint32_t tP = tmem_base + (t == 0 ? Cfg::kColP0 : Cfg::kColP1);
            const uint32_t tO = tmem_base + (t == 0 ? Cfg::kColO0 : Cfg::kColO1);
            const uint32_t bar_s = smem_addr(&sh.s_full[t]);
            const uint32_t bar_ph = smem_addr(&sh.p_half[t]);
            const uint32_t bar_p = smem_addr(&sh.p_full[t]);
            auto desc = [](uint32_t lo) -> uint64_t {
                return (static_cast<uint64_t>(kDescHi) << 32) | lo;
            };
            auto issue_qk = [&](int stage) {
                const uint32_t klo = k_lo0 + stage * (Cfg::kKBytes >> 4);
#pragma unroll
                for (int k = 0; k < DQK / 16; ++k) {
                    const uint32_t koff = ((k / 4) * kChunkBytes + (k % 4) * 32) >> 4;
                    mma_ss(tS, desc(q_lo + koff), desc(klo + koff), kIdescQK, k > 0 ? 1u : 0u);
                }
            };
            // O_t += P_t[:, 64*half .. 64*half+63] V_j[64*half .., :]  (four k-steps of 16 keys)
            auto issue_pv_half = [&](auto hc, int stage, uint32_t accumulate) {
                constexpr int half = decltype(hc)::value;
                const uint32_t vlo = v_lo0 + stage * (Cfg::kVBytes >> 4);
#pragma unroll
                for (int kk = 4 * half; kk < 4 * half + 4; ++kk)
                    mma_ts(tO, tP + kk * 8, desc(vlo + kk * (2048 >> 4)), kIdescPV,
                           (half == 0 && kk == 0) ? accumulate : 1u);
            };
            // The two issuing threads alternate strictly, one block of MMAs each (round r of thread
            // 0, then round r of thread 1, then round r+1 of thread 0, ...), so that the tiles stay
            // half a period apart: the softmax of one tile runs under the MMAs of the other.  All
            // mbarrier waits of a round happen before the thread takes its turn.
            const uint32_t bar_turn_mine = smem_addr(&sh.turn[t]);
            const uint32_t bar_turn_other = smem_addr(&sh.turn[t ^ 1]);
            int round = 0;
            auto take_turn = [&]() -> bool {
                if (t == 0 && round == 0) return true;
                const uint32_t parity = (t == 0) ? ((round - 1) & 1) : (round & 1);
                return mbar_wait(bar_turn_mine, parity, wctx, kSiteMmaTurn);
            };
            auto pass_turn = [&]() { mbar_arrive(bar_turn_other); ++round; };

            bool ok = mbar_wait(smem_addr(&sh.k_full[0]), 0, wctx, kSiteMmaKvFull);
            if (ok && nkv_t > 0) ok = mbar_wait(smem_addr(&sh.q_full[t]), 0, wctx, kSiteMmaQFull);
            ok = ok && take_turn();
            if (ok) {
                if (nkv_t > 0) {
                    tc_fence_after_sync();
                    issue_qk(0);
                    tc_commit(bar_s);
                }
                tc_commit(smem_addr(&sh.k_empty[0]));   // arrives at once if nothing was issued
                pass_turn();
            }
            int sv = 0, sk = (NK > 1) ? 1 : 0;       // stage of V_j and of K_{j+1}
            uint32_t ph_v = 0, ph_k = (NK > 1) ? 0u : 1u;
            for (int j = 0; j < n_max && ok; ++j) {
                const uint32_t bar_ve = smem_addr(&sh.v_empty[sv]);
                const uint32_t bar_ke = smem_addr(&sh.k_empty[sk]);
                // Both threads wait for every stage, also on iterations without work for their
                // tile, so that neither arrives twice in one phase of an "empty" barrier.
                ok = mbar_wait(smem_addr(&sh.v_full[sv]), ph_v, wctx, kSiteMmaKvFull);
                if (ok && j + 1 < n_max) ok = mbar_wait(smem_addr(&sh.k_full[sk]), ph_k, wctx, kSiteMmaKvFull);
                if constexpr (Cfg::kSeparateP) {
                    // Next score block first, outside the alternation: it needs S_t(j) to have been read, not P_t(j).
                    if (ok && j + 1 < nkv_t) {
                        ok = mbar_wait(smem_addr(&sh.s_read[t]), j & 1, wctx, kSiteMmaSFree);
                        if (ok) {
                            tc_fence_after_sync();
                            issue_qk(sk);
                            tc_commit(bar_s);
                        }
                    }
                    if (ok && j + 1 < n_max) tc_commit(bar_ke);   // arrives at once if nothing was issued
                }
                if (ok && j < nkv_t) {
                    FA_TRACE_STAMP(2, j, t * 4 + 0);
                    ok = mbar_wait(bar_ph, j & 1, wctx, kSiteMmaPFull);
                    FA_TRACE_STAMP(2, j, t * 4 + 1);
                }
                ok = ok && take_turn();
                if (!ok) break;
                tc_fence_after_sync();
                if (j < nkv_t) {
                    issue_pv_half(IntC<0>{}, sv, j > 0 ? 1u : 0u);
                    // the other thread has nothing to issue while this tile's softmax is finishing,
                    // so waiting here with the turn in hand costs nothing
                    ok = mbar_wait(bar_p, j & 1, wctx, kSiteMmaPFull);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue_pv_half(IntC<1>{}, sv, 1u);
                    if constexpr (Cfg::kSeparateP) tc_commit(smem_addr(&sh.pv_done[t]));
                    FA_TRACE_STAMP(2, j, t * 4 + 2);
                }
                if (!Cfg::kSeparateP && j + 1 < nkv_t) {
                    issue_qk(sk);
                    tc_commit(bar_s);
                    FA_TRACE_STAMP(2, j, t * 4 + 3);
                } else if (j + 1 == nkv_t) {
                    tc_commit(smem_addr(&sh.o_final[t]));
                }
                tc_commit(bar_ve);
                if (!Cfg::kSeparateP && j + 1 < n_max) tc_commit(bar_ke);
                pass_turn();
                if (++sv == NV) { sv = 0; ph_v ^= 1u; }
                if (++sk == NK) { sk = 0; ph_k ^= 1u; }
            }
        }
    } else if (warp == 14) {
        // ============================================================ TMA loads
        setmaxnreg_dec<kRegsOther>();
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
            // Order of the first requests: Q_0 and K_0 (all the first MMA needs), then Q_1, then V_0.
            // When a whole wave of CTAs starts at once these first loads are HBM-bandwidth-bound.
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
    }

    else {
        setmaxnreg_dec<kRegsOther>();     // idle warp of the fourth warpgroup
    }

    // ---------------------------------------------------------------- teardown (all warps)
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 12) tmem_dealloc(tmem_base, Cfg::kTmemCols);
#ifdef FA_TRACE
    if (warp == 12 && lane == 0 && p.trace) {
        unsigned long long g; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(g));
        long long* rec = p.trace + kTraceRoles * kTraceIters * kTraceEvents + 4ll * blockIdx.x;
        rec[2] = static_cast<long long>(g); rec[3] = n_max;
    }
#endif
}


// Merge of the split-KV partials (Algorithm 2's reduction over the C spatial partitions, in the
// corrected form: every partial is rescaled to the common maximum).  With O_c = G'_c / s_c and
// lse_c = u_c + ln s_c the merged result is lse = ln sum_c exp(lse_c), O = sum_c exp(lse_c - lse) O_c.
// One warp per query row.  The kernel runs behind the attention kernel of a latency-bound launch, so
// it is written for few dependent round trips to memory: the lanes take the C log-sum-exps side by
// side (two passes, reduced with shuffles), then every lane accumulates its four output columns
// with the loads of four partials in flight at a time.
template <int DV>
__global__ void __launch_bounds__(128)
fa_combine_kernel(const float* __restrict__ o_part, const float* __restrict__ lse_part,
                  __nv_bfloat16* __restrict__ O, float* __restrict__ lse,
                  long long n_rows, int n_splits, int Hq, int Sq,
                  long long o_stride_b, long long o_stride_h, long long o_stride_s) {
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();          // the partials come from the kernel before this one
    const long long row = static_cast<long long>(blockIdx.x) * 4 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= n_rows) return;
    const float* lrow = lse_part + row;                 // partial c at lrow[c * n_rows]
    float m = -INFINITY;
    for (int cidx = lane; cidx < n_splits; cidx += 32) m = fmaxf(m, lrow[cidx * n_rows]);
#pragma unroll
    for (int sh = 16; sh > 0; sh >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, sh));
    float denom = 0.f;
    if (m != -INFINITY)
        for (int cidx = lane; cidx < n_splits; cidx += 32) denom += expf(lrow[cidx * n_rows] - m);
#pragma unroll
    for (int sh = 16; sh > 0; sh >>= 1) denom += __shfl_xor_sync(0xffffffffu, denom, sh);
    const float inv = denom > 0.f ? 1.f / denom : 0.f;
    const long long bh = row / Sq;
    __nv_bfloat16* o_row = O + (bh / Hq) * o_stride_b + (bh % Hq) * o_stride_h + (row - bh * Sq) * o_stride_s;
    auto weight = [&](float lc) { return (lc == -INFINITY || m == -INFINITY) ? 0.f : expf(lc - m) * inv; };
#pragma unroll
    for (int col = 0; col < DV; col += 128) {
        if (col + lane * 4 >= DV) break;
        const float* orow = o_part + row * DV + col + lane * 4;     // partial c at orow[c * n_rows * DV]
        const long long step = n_rows * DV;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        int cidx = 0;
        for (; cidx + 4 <= n_splits; cidx += 4) {
            float lc[4];
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                lc[u] = lrow[(cidx + u) * n_rows];
                v[u] = *reinterpret_cast<const float4*>(orow + (cidx + u) * step);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float wgt = weight(lc[u]);
                acc.x = fmaf(wgt, v[u].x, acc.x);
                acc.y = fmaf(wgt, v[u].y, acc.y);
                acc.z = fmaf(wgt, v[u].z, acc.z);
                acc.w = fmaf(wgt, v[u].w, acc.w);
            }
        }
        for (; cidx < n_splits; ++cidx) {
            const float wgt = weight(lrow[cidx * n_rows]);
            const float4 v = *reinterpret_cast<const float4*>(orow + cidx * step);
            acc.x = fmaf(wgt, v.x, acc.x);
            acc.y = fmaf(wgt, v.y, acc.y);
            acc.z = fmaf(wgt, v.z, acc.z);
            acc.w = fmaf(wgt, v.w, acc.w);
        }
        uint2 packed;
        packed.x = ptx::pack_bf16x2(acc.x, acc.y);
        packed.y = ptx::pack_bf16x2(acc.z, acc.w);
        *reinterpret_cast<uint2*>(o_row + col + lane * 4) = packed;
    }
    if (lane == 0 && lse) lse[row] = (m == -INFINITY) ? -INFINITY : m + logf(denom);
}

}  // namespace fa
