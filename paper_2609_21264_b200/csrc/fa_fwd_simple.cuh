// Serialised attention forward kernel for sm_100a: one 128-row query tile per
// CTA, one K/V tile in flight, no overlap between TMA, MMA and softmax.
//
// It runs the per-tile recurrence of Algorithm 1 (score tile, row max, running
// max, exponentials, bf16 P, rescale factor r, G' <- P.V + G'.r, running sum)
// with fp32 state, and divides by the running sum at the end (Section 2.1).
// Both contractions are tcgen05 MMAs with TMEM accumulators; P goes back to
// TMEM as the A operand of the second MMA, so scores never leave the SM.
//
// This variant is the bring-up and cross-check kernel: the pipelined kernel
// must reproduce its results.  It is selectable through the library
// (FA_KERNEL=simple) and is not the one the benchmark times.
#pragma once

#include <math.h>

#include "fa_common.cuh"
#include "ptx.cuh"

namespace fa {

template <int DQK, int DV>
struct SimpleCfg {
    static constexpr int kQChunks = DQK / kChunkCols;
    static constexpr int kVChunks = DV / kChunkCols;
    static constexpr int kQBytes = kQChunks * kChunkBytes;
    static constexpr int kKBytes = kQBytes;
    static constexpr int kVBytes = kVChunks * kChunkBytes;
    // TMEM columns: S (128 fp32) | O (DV fp32) | P (64 x bf16x2)
    static constexpr int kColS = 0;
    static constexpr int kColO = 128;
    static constexpr int kColP = 128 + DV;
    static constexpr int kTmemCols = (128 + DV + 64) <= 256 ? 256 : 512;
    static constexpr int kSmemBytes = kQBytes + kKBytes + kVBytes + 1024;   // + alignment slack
};

template <int DQK, int DV>
__global__ void __launch_bounds__(128, 1)
fa_fwd_simple_kernel(const __grid_constant__ CUtensorMap tm_q,
                     const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v,
                     const FwdParams p) {
    using Cfg = SimpleCfg<DQK, DV>;
    using namespace ptx;

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[4];   // 0: Q, 1: K, 2: V, 3: MMA done
    __shared__ uint32_t tmem_base_slot;
    __shared__ uint32_t abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;

    const uint32_t smem_base = (smem_addr(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + Cfg::kQBytes;
    const uint32_t sV = sK + Cfg::kKBytes;
    const uint32_t bar_q = smem_addr(&bars[0]);
    const uint32_t bar_k = smem_addr(&bars[1]);
    const uint32_t bar_v = smem_addr(&bars[2]);
    const uint32_t bar_mma = smem_addr(&bars[3]);

    const int q_tile = static_cast<int>(gridDim.x) - 1 - static_cast<int>(blockIdx.x);  // heavy tiles first
    const int hq = blockIdx.y;
    const int b = blockIdx.z;
    const int kvh = hq / (p.Hq / p.Hkv);
    const int i0 = q_tile * kTileM;
    const int q_idx = b * p.Hq + hq;
    // fixed-length batch, or sequence b of a packed variable-length batch
    int Sq = p.Sq, Sk = p.Sk, q_row0 = 0, k_row0 = 0, tb = b;
    size_t lse_row0 = static_cast<size_t>(q_idx) * p.Sq;
    long long o_base = b * p.o_stride_b + hq * p.o_stride_h;
    if (p.cu_q) {
        q_row0 = p.cu_q[b];
        k_row0 = p.cu_k[b];
        Sq = p.cu_q[b + 1] - q_row0;
        Sk = p.cu_k[b + 1] - k_row0;
        tb = 0;
        lse_row0 = static_cast<size_t>(hq) * p.total_q + q_row0;
        o_base = q_row0 * p.o_stride_s + hq * p.o_stride_h;
    }
    if (i0 >= Sq) return;      // whole CTA, before any set-up
    const int off = Sk - Sq;
    const int n_kv = kv_tiles_for_q_tile(i0, kTileM, Sq, Sk, p.causal);

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(bar_q, 1);
        mbar_init(bar_k, 1);
        mbar_init(bar_v, 1);
        mbar_init(bar_mma, 1);
        fence_mbar_init();
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
    }
    if (warp == 0) {
        tmem_alloc(smem_addr(&tmem_base_slot), Cfg::kTmemCols);
        tmem_relinquish_alloc_permit();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();

    const uint32_t tmem_base = tmem_base_slot;
    const uint32_t lane_sel = static_cast<uint32_t>(warp * 32) << 16;
    const uint32_t tS = tmem_base + Cfg::kColS;
    const uint32_t tO = tmem_base + Cfg::kColO;
    const uint32_t tP = tmem_base + Cfg::kColP;

    WaitCtx wctx{&abort_flag, p.status, p.wait_limit_ns};

    constexpr uint32_t kIdescQK = make_idesc_bf16_f32(kTileM, kTileN, false, false);
    constexpr uint32_t kIdescPV = make_idesc_bf16_f32(kTileM, DV, false, true);

    const int i_glob = i0 + tid;                 // this thread's query row
    int kmax_row = Sk - 1;                       // last visible key of this row
    if (p.causal && i_glob + off < kmax_row) kmax_row = i_glob + off;

    float m_run = -INFINITY;   // running row max (log2 units)
    float l_run = 0.f;         // running row sum
    uint32_t ph_kv = 0, ph_mma = 0;
    bool ok = true;

    if (tid == 0 && n_kv > 0) {
        mbar_arrive_expect_tx(bar_q, Cfg::kQBytes);
#pragma unroll
        for (int c = 0; c < Cfg::kQChunks; ++c)
            tma_load_4d(sQ + c * kChunkBytes, &tm_q, bar_q, c * kChunkCols, q_row0 + i0, hq, tb);
    }

    for (int j = 0; j < n_kv && ok; ++j) {
        const int j0 = j * kTileN;
        if (tid == 0) {
            mbar_arrive_expect_tx(bar_k, Cfg::kKBytes);
#pragma unroll
            for (int c = 0; c < Cfg::kQChunks; ++c)
                tma_load_4d(sK + c * kChunkBytes, &tm_k, bar_k, c * kChunkCols, k_row0 + j0, kvh, tb);
            mbar_arrive_expect_tx(bar_v, Cfg::kVBytes);
#pragma unroll
            for (int c = 0; c < Cfg::kVChunks; ++c)
                tma_load_4d(sV + c * kChunkBytes, &tm_v, bar_v, c * kChunkCols, k_row0 + j0, kvh, tb);

            bool w = true;
            if (j == 0) w = mbar_wait(bar_q, 0, wctx, kSiteSimpleQ);
            w = w && mbar_wait(bar_k, ph_kv, wctx, kSiteSimpleK);
            if (w) {
                tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < DQK / 16; ++k) {
                    const uint32_t koff = (k / 4) * kChunkBytes + (k % 4) * 32;
                    const uint64_t a = make_smem_desc_sw128(sQ + koff, 16, 1024);
                    const uint64_t bd = make_smem_desc_sw128(sK + koff, 16, 1024);
                    mma_ss(tS, a, bd, kIdescQK, k > 0 ? 1u : 0u);
                }
                tc_commit(bar_mma);
            }
        }
        ok = mbar_wait(bar_mma, ph_mma, wctx, kSiteSimpleMma);
        ph_mma ^= 1;
        if (!ok) break;
        tc_fence_after_sync();

        // ---- online softmax on this thread's row (Algorithm 1: max, running max, exp, bf16 P)
        const bool need_mask = (j0 + kTileN - 1 > kmax_row);
        float mx = -INFINITY;
#pragma unroll 1
        for (int c4 = 0; c4 < 4; ++c4) {
            uint32_t r[32];
            tmem_ld_x32(tS + lane_sel + c4 * 32, r);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                float x = __uint_as_float(r[e]) * p.scale_log2;
                if (need_mask && (j0 + c4 * 32 + e > kmax_row)) x = -INFINITY;
                mx = fmaxf(mx, x);
            }
        }
        const float m_new = fmaxf(m_run, mx);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = exp2_approx(m_run - m_use);   // r = exp(u' - u)
        float rowsum = 0.f;
#pragma unroll 1
        for (int c4 = 0; c4 < 4; ++c4) {
            uint32_t r[32];
            tmem_ld_x32(tS + lane_sel + c4 * 32, r);
            tc_wait_ld();
            uint32_t pk[16];
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
                float x0 = __uint_as_float(r[e]) * p.scale_log2;
                float x1 = __uint_as_float(r[e + 1]) * p.scale_log2;
                if (need_mask) {
                    if (j0 + c4 * 32 + e > kmax_row) x0 = -INFINITY;
                    if (j0 + c4 * 32 + e + 1 > kmax_row) x1 = -INFINITY;
                }
                const float p0 = exp2_approx(x0 - m_use);
                const float p1 = exp2_approx(x1 - m_use);
                rowsum += p0 + p1;
                pk[e / 2] = pack_bf16x2(p0, p1);
            }
            tmem_st_x16(tP + lane_sel + c4 * 16, pk);
        }
        l_run = l_run * alpha + rowsum;
        m_run = m_new;

        // ---- rescale the accumulator (G' <- G' . r) when any row of the warp moved its max
        if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll 1
            for (int c = 0; c < DV / 32; ++c) {
                uint32_t r[32];
                tmem_ld_x32(tO + lane_sel + c * 32, r);
                tc_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                tmem_st_x32(tO + lane_sel + c * 32, r);
            }
        }
        tc_wait_st();
        tc_fence_before_sync();
        __syncthreads();

        // ---- G' += P . V_j
        if (tid == 0) {
            if (mbar_wait(bar_v, ph_kv, wctx, kSiteSimpleV)) {
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < kTileN / 16; ++kk) {
                    const uint64_t bd = make_smem_desc_sw128(sV + kk * 2048, kChunkBytes, 1024);
                    mma_ts(tO, tP + kk * 8, bd, kIdescPV, (j > 0 || kk > 0) ? 1u : 0u);
                }
                tc_commit(bar_mma);
            }
        }
        ph_kv ^= 1;
        ok = mbar_wait(bar_mma, ph_mma, wctx, kSiteSimpleMma);
        ph_mma ^= 1;
        if (!ok) break;
        tc_fence_after_sync();
    }

    // ---- epilogue: O = G' / s (bf16), lse = ln2 * u + ln s
    if (ok && i_glob < Sq) {
        __nv_bfloat16* o_row = p.O + (o_base + static_cast<long long>(i_glob) * p.o_stride_s);
        const bool empty = (n_kv == 0) || !(l_run > 0.f);
        if (p.lse && tid < kTileM) {
            p.lse[lse_row0 + i_glob] =
                empty ? -INFINITY : (m_run * 0.6931471805599453f + logf(l_run));
        }
        if (n_kv == 0) {
            const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int c = 0; c < DV / 8; ++c) reinterpret_cast<uint4*>(o_row)[c] = z;
        }
    }
    if (ok && n_kv > 0) {
        const float inv_l = (l_run > 0.f) ? (1.f / l_run) : 0.f;
#pragma unroll 1
        for (int c = 0; c < DV / 32; ++c) {
            uint32_t r[32];
            tmem_ld_x32(tO + lane_sel + c * 32, r);   // warp-collective: all lanes take part
            tc_wait_ld();
            if (i_glob < Sq) {
                __nv_bfloat16* o_row = p.O + (o_base + static_cast<long long>(i_glob) * p.o_stride_s);
                uint32_t pk[16];
#pragma unroll
                for (int e = 0; e < 32; e += 2)
                    pk[e / 2] = pack_bf16x2(__uint_as_float(r[e]) * inv_l,
                                            __uint_as_float(r[e + 1]) * inv_l);
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    reinterpret_cast<uint4*>(o_row + c * 32)[v] =
                        make_uint4(pk[4 * v], pk[4 * v + 1], pk[4 * v + 2], pk[4 * v + 3]);
            }
        }
    }

    // ---- teardown: every thread arrives here, also after a failed wait
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, Cfg::kTmemCols);
}

}  // namespace fa
