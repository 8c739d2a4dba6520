// Block-scaled 8-bit variant of the pipelined attention forward kernel for sm_100a.
//
// The paper's second device computes its contractions in a block floating-point format (groups
// of values sharing one exponent) instead of bf16 (Section 3, data types).  The counterpart on
// this hardware: Q, K and V are stored as e4m3 with one fp32 scale per block, and both
// contractions run on the 8-bit tensor-core path (tcgen05.mma kind::f8f6f4, fp32 accumulation in
// TMEM), which has twice the bf16 rate and half the operand traffic.
//   * Q: one scale per 128-row query tile and head, K: one scale per 128-row key tile and K/V
//     head.  A score tile is then S = (sq * sk_j) * (Q8 K8_j^T), and since the softmax already
//     multiplies every score by scale * log2 e inside the exp2 argument, the block scales are
//     folded into that constant, tile by tile, at no cost.
//   * V: one scale per K/V head.  O accumulates over key tiles inside TMEM, so a per-tile scale
//     would have to be folded into P before its rounding to e4m3, which costs precision for
//     tiles with small values; the per-head scale is applied once, with 1/s, in the epilogue.
//   * P is rounded to e4m3 (four values per 32-bit TMEM column) before the second contraction;
//     the row sums use the unrounded fp32 values, as in the bf16 kernel.
// Everything else (roles, barriers, the two-tile schedule, lazy reference maximum kept in scaled
// log2 units, bounded waits, TMA-store epilogue, dependent launch) is the bf16 kernel's; read
// fa_fwd_pipelined.cuh first.  Head sizes 64 and 128, fixed-length contiguous [B,H,S,d] tensors, no
// split-KV.  O is bf16, lse fp32.
// TMEM: S_0 [0,128) S_1 [128,256) O_0 [256,384) O_1 [384,512); e4m3 P_t overlays S_t[0,32).
#pragma once

#include <math.h>

#include "fa_common.cuh"
#include "fa_fwd_pipelined.cuh"
#include "ptx.cuh"

namespace fa {

// D = head size of Q/K and of V: 128 (rows of 128 bytes, 128-byte swizzle) or 64 (rows of 64 bytes,
// 64-byte swizzle: 8-row groups 512 bytes apart, a 32-key step of V 2048 bytes).
template <int D>
struct Fp8Cfg {
    static_assert(D == 64 || D == 128, "head sizes of the 8-bit kernels");
    static constexpr int kD = D;
    static constexpr int kTileBytes8 = kTileM * kD;      // one 128 x D e4m3 tile (16 or 8 KB), one swizzled chunk
    static constexpr int kOBytes = (D / kChunkCols) * kChunkBytes;      // bf16 output tile (64-column chunks)
    static constexpr int kKStages = (D == 128) ? 3 : 4;
    static constexpr int kVStages = (D == 128) ? 3 : 4;
    // descriptor high word: stride between 8-row groups, version, swizzle mode
    static constexpr uint32_t kDescHi = ((D == 128 ? 1024u : 512u) >> 4) | (1u << 14) | ((D == 128 ? 2u : 4u) << 29);
    static constexpr uint32_t kVStep = (32u * D) >> 4;   // 32 keys of V, in descriptor address units
    // Q_0, Q_1, the K and V rings, and one staging buffer per query tile for the bf16 output
    static constexpr int kSmemTiles = (2 + kKStages + kVStages) * kTileBytes8 + 2 * kOBytes;
    static constexpr int kTmemCols = 512;
    static constexpr int kColS0 = 0, kColS1 = 128, kColO0 = 256, kColO1 = 384;
    static constexpr int kThreads = 512;
};

// Share of the exponentials of the 8-bit kernels that is computed on the FMA pipe: every kFp8EmuEvery-th pair (0 = none).
// Measured on B200 with Gaussian data (pair kernel, TFLOP/s, none / every 4th / 3rd / 2nd pair): causal S 2048 921 / 1033 /
// 1029 / 966, B4 S 8192 1270 / 1377 / 1384 / 1303, S 32768 1422 / 1519 / 1546 / 1408, 64-round non-causal items 1321 /
// 1611 / 1540 / 1402.
#ifndef FA_FP8_EMU_EVERY
#define FA_FP8_EMU_EVERY 4
#endif
constexpr int kFp8EmuEvery = FA_FP8_EMU_EVERY;

struct Fp8Params {
    const float* q_scale;    // [B, Hq, n_q_tiles] or nullptr (= 1)
    const float* k_scale;    // [B, Hkv, n_kv_tiles] or nullptr
    const float* v_scale;    // [B, Hkv] or nullptr
    int n_kv_tiles;          // ceil(Sk / 128)
    // MX variant (e8m0 scales per 32 elements along the contraction; fa_fwd_fp8_stream_kernel with kMx): one
    // 512-byte scale atom per 128-row tile, byte (r % 32) * 16 + (r / 32) * 4 + kb
    const uint8_t* q_sf;     // [B, Hq, n_q_tiles, 512]: row r of the query tile, block kb of its d columns
    const uint8_t* k_sf;     // [B, Hkv, n_kv_tiles, 512]: key r of the K tile, block kb of its d columns
    const uint8_t* v_sf;     // [B, Hkv, n_kv_tiles, 512]: column r of V, block kb of the tile's 128 keys
};

template <int D>
constexpr int fp8_smem_bytes() { return Fp8Cfg<D>::kSmemTiles + static_cast<int>(sizeof(PipeShared)); }

// kHeadPair: the two query tiles are the same query tile of two adjacent heads of a K/V group, as in
// fa_fwd_pipelined_kernel.
template <int D, bool kHeadPair = false>
__global__ void __launch_bounds__(512, 1)
fa_fwd_fp8_kernel(const __grid_constant__ CUtensorMap tm_q,
                  const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v,
                  const __grid_constant__ CUtensorMap tm_o,
                  const FwdParams p, const Fp8Params f) {
    using Cfg = Fp8Cfg<D>;
    using namespace ptx;
    constexpr int NK = Cfg::kKStages;
    constexpr int NV = Cfg::kVStages;
    constexpr int DV = Cfg::kD;
    constexpr int kTile8 = Cfg::kTileBytes8;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    PipeShared& sh = *reinterpret_cast<PipeShared*>(smem_raw + Cfg::kSmemTiles);

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
    const uint32_t sK = sQ + 2 * kTile8;                         // NK stages
    const uint32_t sV = sK + NK * kTile8;                        // NV stages
    const uint32_t sStage = sV + NV * kTile8;                    // bf16 output tiles pass through here (one buffer per tile)

    // grid order: see the bf16 kernel (L2-sized head groups, longest-first inside a group)
    const int n_pairs = kHeadPair ? p.n_q_tiles : (p.n_q_tiles + 1) / 2;
    const int n_bh = p.B * p.Hq;
    const int item = static_cast<int>(blockIdx.x);
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
    const int kv_idx = b * p.Hkv + kvh;
    const int off = p.Sk - p.Sq;

    const int i0_0 = (kHeadPair ? pair : 2 * pair) * kTileM, i0_1 = kHeadPair ? i0_0 : i0_0 + kTileM;
    auto own_tiles = [&](int i0) -> int {
        if (i0 >= p.Sq) return 0;
        return kv_tiles_for_q_tile(i0, kTileM, p.Sq, p.Sk, p.causal);
    };
    const int nkv_0 = own_tiles(i0_0);
    const int nkv_1 = own_tiles(i0_1);
    const int n_max = nkv_0 > nkv_1 ? nkv_0 : nkv_1;

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
    grid_dependency_wait();

    const uint32_t tmem_base = sh.tmem_base;
    WaitCtx wctx{&sh.abort_flag, p.status, p.wait_limit_ns};

    if (warp < 8) {
        // ============================================================ softmax of tile t
        setmaxnreg_inc<kRegsSoftmax>();
        const int t = warp >> 2;
        const int row = tid & (kTileM - 1);
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + (t == 0 ? Cfg::kColS0 : Cfg::kColS1) + lane_sel;
        const uint32_t bar_s = smem_addr(&sh.s_full[t]);
        const uint32_t bar_p = smem_addr(&sh.p_full[t]);
        const uint32_t bar_ph = smem_addr(&sh.p_half[t]);
        const uint32_t bar_scale = smem_addr(&sh.scale_full[t]);
        const int i0_t = t == 0 ? i0_0 : i0_1;
        const int hq_t = kHeadPair ? hq + t : hq;          // query head of this tile
        const int q_idx_t = kHeadPair ? q_idx + t : q_idx;
        const int nkv_t = t == 0 ? nkv_0 : nkv_1;
        const int i_glob = i0_t + row;
        int kmax_row = p.Sk - 1;
        if (p.causal && i_glob + off < kmax_row) kmax_row = i_glob + off;
        // scale * log2 e * (scale of this query tile); the key tile's scale joins per iteration
        const float cq = p.scale_log2 *
                         ((f.q_scale && i0_t < p.Sq) ? __ldg(f.q_scale + static_cast<size_t>(q_idx_t) * p.n_q_tiles + (i0_t / kTileM)) : 1.f);
        const float* k_scale = f.k_scale ? f.k_scale + static_cast<size_t>(kv_idx) * f.n_kv_tiles : nullptr;
        float sk_next = (k_scale && nkv_t > 0) ? __ldg(k_scale) : 1.f;

        float m_ref = -INFINITY;   // reference maximum in scaled log2 units (block scales differ per tile)
        float l = 0.f;
        bool ok = true;
        for (int j = 0; j < nkv_t; ++j) {
            const float c = cq * sk_next;                  // exp2 argument = raw score * c - m_ref
            if (k_scale && j + 1 < nkv_t) sk_next = __ldg(k_scale + j + 1);
            ok = __all_sync(0xffffffffu, mbar_wait(bar_s, j & 1, wctx, kSiteSoftmaxSFull));
            if (!ok) break;
            tc_fence_after_sync();
            const int j0 = j * kTileN;
            const bool need_mask = (j0 + kTileN - 1 > kmax_row);

            const float2 c2 = make_float2(c, c);
            float2 nmc2;
            float2 sum_a = make_float2(0.f, 0.f), sum_b = make_float2(0.f, 0.f);
            float alpha = 1.f;
            uint32_t s[kTileN];
            // With 8-bit operands the MMAs of a tile take half the cycles of the exponentials (512 against 1024 on the
            // MUFU at 16 per cycle and SM): the loop is MUFU-bound.  Every kFp8EmuEvery-th pair of exponentials therefore
            // goes to the FMA pipe (ptx::exp2_poly2, relative error 7.5e-5 against e4m3's 2^-4 for P and 1e-3 for lse).
            auto exp_chunk = [&](int q) {
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[q * 32 + e]),
                                                            __uint_as_float(s[q * 32 + e + 1])), c2, nmc2);
                    if (kFp8EmuEvery > 0 && ((e / 2) % (kFp8EmuEvery > 0 ? kFp8EmuEvery : 1)) == kFp8EmuEvery - 1) {
                        const float2 r = exp2_poly2(x);
                        s[q * 32 + e] = __float_as_uint(r.x);
                        s[q * 32 + e + 1] = __float_as_uint(r.y);
                    } else {
                        s[q * 32 + e] = __float_as_uint(exp2_approx(x.x));
                        s[q * 32 + e + 1] = __float_as_uint(exp2_approx(x.y));
                    }
                }
            };
            // Row sum (of the unrounded values), e4m3 conversion and store of one 32-key chunk of P.
            auto emit_chunk = [&](int q) {
                uint32_t pk[8];
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    const float2 v0 = make_float2(__uint_as_float(s[q * 32 + e]), __uint_as_float(s[q * 32 + e + 1]));
                    const float2 v1 = make_float2(__uint_as_float(s[q * 32 + e + 2]), __uint_as_float(s[q * 32 + e + 3]));
                    sum_a = __fadd2_rn(sum_a, v0);
                    sum_b = __fadd2_rn(sum_b, v1);
                    pk[e / 4] = pack_e4m3x4(v0.x, v0.y, v1.x, v1.y);
                }
                tmem_st_x8(tS + q * 8, pk);
            };
#pragma unroll 1
            for (;;) {
                tmem_ld_x32(tS + 0, s + 0);
                tmem_ld_x32(tS + 32, s + 32);
                tmem_ld_x32(tS + 64, s + 64);
                tmem_ld_x32(tS + 96, s + 96);
                tc_wait_ld();
                if (need_mask) {
#pragma unroll
                    for (int e = 0; e < kTileN; ++e)
                        if (j0 + e > kmax_row) s[e] = 0xff800000u;   // -inf
                }
                const float mc = (m_ref == -INFINITY) ? 0.f : m_ref;
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
                mx = fmax3(mx, a[6], a[7]) * c;                // c > 0: the maximum commutes with the scaling
                const bool grow = mx > m_ref + kRescaleThresholdLog2;
                if (!__any_sync(0xffffffffu, grow)) break;
                if (grow) {
                    alpha = exp2_approx(m_ref - mx);           // r = exp(u' - u); 0 on the first tile
                    m_ref = mx;
                }
            }
            sh.alpha[t][j & 1][row] = alpha;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_scale);

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
            tc_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_p);
        }
        // epilogue: O = sv * G' / s (bf16), lse = u + ln s
        if (ok && i0_t < p.Sq) {
            const size_t lse_row0 = static_cast<size_t>(q_idx_t) * p.Sq;
            if (nkv_t == 0) {         // no key visible to any row of this tile
                if (i_glob < p.Sq) {
                    __nv_bfloat16* o_row = p.O + (b * p.o_stride_b + hq_t * p.o_stride_h +
                                                  static_cast<long long>(i_glob) * p.o_stride_s);
                    const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int v = 0; v < DV / 8; ++v) reinterpret_cast<uint4*>(o_row)[v] = z;
                    if (p.lse) p.lse[lse_row0 + i_glob] = -INFINITY;
                }
            } else if (__all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.o_final[t]), 0, wctx, kSiteEpiOFull))) {
                tc_fence_after_sync();
                const float sv = f.v_scale ? __ldg(f.v_scale + kv_idx) : 1.f;
                const float inv_l = (l > 0.f) ? (sv / l) : 0.f;
                if (p.lse && i_glob < p.Sq)
                    p.lse[lse_row0 + i_glob] = (l > 0.f) ? (m_ref * 0.6931471805599453f + logf(l)) : -INFINITY;
                const uint32_t tO = tmem_base + (t == 0 ? Cfg::kColO0 : Cfg::kColO1) + lane_sel;
                const uint32_t sO = sStage + t * Cfg::kOBytes + row * 128;
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
                    mbar_wait(smem_addr(&sh.o_staged[t]), 0, wctx, kSiteEpiStaged)) {
#pragma unroll
                    for (int ch = 0; ch < DV / kChunkCols; ++ch)
                        tma_store_4d(&tm_o, sStage + t * Cfg::kOBytes + ch * kChunkBytes, ch * kChunkCols, i0_t, hq_t, b);
                    tma_store_commit();
                    tma_store_wait_read_all();     // the CTA's shared memory outlives the reads
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
            }
        }
    } else if (warp == 12 || warp == 13) {
        // ============================================================ MMA issue for tile t = warp - 12
        setmaxnreg_dec<kRegsOther>();
        if (elect_one() && n_max > 0) {
            const int t = warp - 12;
            const int nkv_t = (t == 0) ? nkv_0 : nkv_1;
            constexpr uint32_t kIdescQK = make_idesc_e4m3_f32(kTileM, kTileN, false, false);
            constexpr uint32_t kIdescPV = make_idesc_e4m3_f32(kTileM, DV, false, true);
            constexpr uint32_t kDescHi = Cfg::kDescHi;
            // an e4m3 row of D elements is exactly one swizzled row of D bytes: a tile is one chunk
            const uint32_t q_lo = (((sQ + t * kTile8) & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t v_lo0 = ((sV & 0x3FFFFu) >> 4) | ((16384u >> 4) << 16);   // one swizzled row spans dv: the chunk stride is not used
            const uint32_t tS = tmem_base + (t == 0 ? Cfg::kColS0 : Cfg::kColS1);   // P_t overlays it
            const uint32_t tO = tmem_base + (t == 0 ? Cfg::kColO0 : Cfg::kColO1);
            const uint32_t bar_s = smem_addr(&sh.s_full[t]);
            const uint32_t bar_ph = smem_addr(&sh.p_half[t]);
            const uint32_t bar_p = smem_addr(&sh.p_full[t]);
            auto desc = [](uint32_t lo) -> uint64_t {
                return (static_cast<uint64_t>(kDescHi) << 32) | lo;
            };
            // S_t = Q_t K_j^T: D / 32 k-steps of 32 elements (32 bytes along the swizzled row)
            auto issue_qk = [&](int stage) {
                const uint32_t klo = k_lo0 + stage * (kTile8 >> 4);
#pragma unroll
                for (int k = 0; k < Cfg::kD / 32; ++k)
                    mma_ss_f8(tS, desc(q_lo + k * 2), desc(klo + k * 2), kIdescQK, k > 0 ? 1u : 0u);
            };
            // O_t += P_t[:, 64*half .. 64*half+63] V_j[64*half .., :]: two k-steps of 32 keys
            // (8 TMEM columns of P, 32 rows of D bytes of V)
            auto issue_pv_half = [&](auto hc, int stage, uint32_t accumulate) {
                constexpr int half = decltype(hc)::value;
                const uint32_t vlo = v_lo0 + stage * (kTile8 >> 4);
#pragma unroll
                for (int kk = 2 * half; kk < 2 * half + 2; ++kk)
                    mma_ts_f8(tO, tS + kk * 8, desc(vlo + kk * Cfg::kVStep), kIdescPV,
                              (half == 0 && kk == 0) ? accumulate : 1u);
            };
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
            int sv = 0, sk = 1;                      // stage of V_j and of K_{j+1}
            uint32_t ph_v = 0, ph_k = 0;
            for (int j = 0; j < n_max && ok; ++j) {
                const uint32_t bar_ve = smem_addr(&sh.v_empty[sv]);
                const uint32_t bar_ke = smem_addr(&sh.k_empty[sk]);
                ok = mbar_wait(smem_addr(&sh.v_full[sv]), ph_v, wctx, kSiteMmaKvFull);
                if (ok && j + 1 < n_max) ok = mbar_wait(smem_addr(&sh.k_full[sk]), ph_k, wctx, kSiteMmaKvFull);
                if (ok && j < nkv_t) ok = mbar_wait(bar_ph, j & 1, wctx, kSiteMmaPFull);
                ok = ok && take_turn();
                if (!ok) break;
                tc_fence_after_sync();
                if (j < nkv_t) {
                    issue_pv_half(IntC<0>{}, sv, j > 0 ? 1u : 0u);
                    ok = mbar_wait(bar_p, j & 1, wctx, kSiteMmaPFull);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue_pv_half(IntC<1>{}, sv, 1u);
                }
                if (j + 1 < nkv_t) {
                    issue_qk(sk);
                    tc_commit(bar_s);
                } else if (j + 1 == nkv_t) {
                    tc_commit(smem_addr(&sh.o_final[t]));
                }
                tc_commit(bar_ve);
                if (j + 1 < n_max) tc_commit(bar_ke);
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
                mbar_arrive_expect_tx(bar, kTile8);
                tma_load_4d(sQ + t * kTile8, &tm_q, bar, 0, t == 0 ? i0_0 : i0_1, kHeadPair ? hq + t : hq, b);
            };
            load_q(0);
            bool ok = true;
            for (int j = 0; j < n_max && ok; ++j) {
                const int j0 = j * kTileN;
                {
                    const int s = j % NK;
                    ok = mbar_wait(smem_addr(&sh.k_empty[s]), ((j / NK) & 1) ^ 1, wctx, kSiteLoadKvEmpty);
                    if (!ok) break;
                    const uint32_t bar = smem_addr(&sh.k_full[s]);
                    mbar_arrive_expect_tx(bar, kTile8);
                    tma_load_4d(sK + s * kTile8, &tm_k, bar, 0, j0, kvh, b);
                    if (j == 0) load_q(1);
                }
                if (!(p.debug_drop_v_load && j == 0)) {       // (test hook: see FA_FLAG_DEBUG_DROP_V_LOAD)
                    const int s = j % NV;
                    ok = mbar_wait(smem_addr(&sh.v_empty[s]), ((j / NV) & 1) ^ 1, wctx, kSiteLoadKvEmpty);
                    if (!ok) break;
                    const uint32_t bar = smem_addr(&sh.v_full[s]);
                    mbar_arrive_expect_tx(bar, kTile8);
                    tma_load_4d(sV + s * kTile8, &tm_v, bar, 0, j0, kvh, b);
                }
            }
        }
    } else {
        setmaxnreg_dec<kRegsOther>();     // idle warp of the fourth warpgroup
    }

    // ---------------------------------------------------------------- teardown (all warps)
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 12) tmem_dealloc(tmem_base, Cfg::kTmemCols);
}

}  // namespace fa
