// Attention forward kernel for sm_100a: one 128-row query tile per CTA, its K/V tiles streamed
// through two softmax warpgroups that take alternate K/V tiles.
//
// Same arithmetic as fa_fwd_pipelined.cuh (Algorithm 1 with fp32 state, lazy reference maximum,
// bf16 P, one division at the end; read that file first).  What changes is what the two softmax
// warpgroups share.  There they own one query tile each and TMEM is full (2 x (S + O)), so the
// probabilities have to overlay the scores and a tile's next score MMA waits for its P V MMA: a
// K/V tile costs a tile the whole chain softmax -> PV -> QK.  Here the CTA has ONE query tile:
//   TMEM  S^0 [0,128)  S^1 [128,256)  O [256,384)  P^0 [384,448)  P^1 [448,512)
// Warpgroup b = j mod 2 runs the softmax of K/V tile j from S^b into P^b.  The score MMA of tile
// j+2 is issued as soon as S^b has been read into registers, the PV MMA of tile j whenever P^b
// is ready, both off the softmax's path, so the two warpgroups run back to back and side by
// side and the loop is bound by the MUFU/issue rate of the softmax and by the tensor pipe
// instead of by the length of a dependency chain.  The price: K and V tiles are fetched once
// per query tile instead of once per pair (L2 -> shared-memory traffic doubles, about a third of
// the L2's bandwidth), and a CTA's fixed cost is spread over half the work.
//
// The row state (reference maximum u, and every rescale factor r) is handed from one
// warpgroup to the other through shared memory once per K/V tile; each warpgroup keeps its
// own partial row sum and applies every r to it.  Roles:
//   warps 0-3, 4-7  softmax of the even / odd K/V tiles (one query row per thread)
//   warps 8-11      correction: O *= r when the reference maximum moved
//   warp 12         score MMAs (one thread), warp 13: PV MMAs (one thread)
//   warp 14         TMA loads of Q and K, warp 15: TMA loads of V
// Split-KV as in the pair kernel: partials to scratch, merged by fa_combine_kernel.
#pragma once

#include "fa_fwd_pipelined.cuh"

namespace fa {

template <int DQK, int DV>
struct StreamCfg {
    using Base = PipeCfg<DQK, DV>;
    static constexpr int kQChunks = Base::kQChunks;
    static constexpr int kVChunks = Base::kVChunks;
    static constexpr int kQBytes = Base::kQBytes;
    static constexpr int kKBytes = Base::kKBytes;
    static constexpr int kVBytes = Base::kVBytes;
    static constexpr int kKStages = (DQK == 192) ? 2 : 3;
    static constexpr int kVStages = (DQK == 192) ? 2 : 3;
    static constexpr int kTileBytes = kQBytes + kKStages * kKBytes + kVStages * kVBytes;
    static constexpr int kTmemCols = 512;
    static constexpr int kColS = 0;        // S^b at kColS + 128 b
    static constexpr int kColO = 256;
    static constexpr int kColP = 384;      // P^b at kColP + 64 b
    static constexpr int kThreads = 512;
};

struct StreamShared {
    uint64_t q_full;
    uint64_t k_full[4], k_empty[4];
    uint64_t v_full[4], v_empty[4];
    uint64_t s_full[2];      // score MMA -> softmax b: S^b(j) is in TMEM
    uint64_t s_free[2];      // softmax b -> score MMA: S^b(j) is in registers
    uint64_t st_full[2];     // softmax b -> the other warpgroup and correction: u and r of tile j published
    uint64_t p_ready[2];     // softmax b + correction -> PV MMA: P^b(j) written, O rescaled
    uint64_t p_free[2];      // PV MMA -> softmax b, correction: PV(j) complete
    uint64_t o_final;        // PV MMA -> epilogue
    uint64_t l_ready;        // softmax warps -> epilogue: partial row sums published
    uint64_t o_staged;       // softmax warps -> storing thread
    float alpha[2][kTileM];  // r of tile j in slot j & 1
    float mref[kTileM];      // u after the last published tile (raw score units)
    float lsum[2][kTileM];   // final partial row sums of the two warpgroups
    uint32_t tmem_base;
    uint32_t abort_flag;
};

template <int DQK, int DV>
constexpr int stream_smem_bytes() {
    return StreamCfg<DQK, DV>::kTileBytes + static_cast<int>(sizeof(StreamShared));
}

// kVarlen = packed variable-length batch, as in the pair kernel.
// kPack = the query tile holds the (at most 64) query rows of SEVERAL query heads that share one
// K/V head (grouped-query attention with few queries per sequence, as when decoding): row
// h * Sq + i of the tile is query i of the CTA's h-th head.  Every K/V tile is then read and
// multiplied once for p.pack_heads heads instead of once per head.  The tensor maps of Q and
// O have a box of Sq rows x pack_heads heads for it.
template <int DQK, int DV, bool kVarlen = false, bool kPack = false>
__global__ void __launch_bounds__(512, 1)
fa_fwd_stream_kernel(const __grid_constant__ CUtensorMap tm_q,
                     const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v,
                     const __grid_constant__ CUtensorMap tm_o,
                     const FwdParams p) {
    using Cfg = StreamCfg<DQK, DV>;
    using namespace ptx;
    constexpr int NK = Cfg::kKStages;
    constexpr int NV = Cfg::kVStages;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    StreamShared& sh = *reinterpret_cast<StreamShared*>(smem_raw + Cfg::kTileBytes);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    grid_launch_dependents();
    if constexpr (kVarlen) grid_dependency_wait();    // the sequence offsets are read right away

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
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + Cfg::kQBytes;
    const uint32_t sV = sK + NK * Cfg::kKBytes;

    // 1-D grid: L2-sized groups of (batch, head) instances one after the other; inside a group
    // every head's last (with a causal mask: heaviest) query tile first.
    const int n_bh = p.B * p.Hq;
    // With split-KV the C CTAs that share a query tile and take disjoint ranges of its K/V tiles are
    // adjacent in the grid; each writes a normalised fp32 partial that the combine kernel merges.
    const int item = static_cast<int>(blockIdx.x) / p.kv_splits;
    const int split = static_cast<int>(blockIdx.x) - item * p.kv_splits;
    int q_tile = 0, hq, b;
    if constexpr (kPack) {
        // one item per pack of heads; all items are equally long
        const int packs = p.Hq / p.pack_heads;
        b = item / packs;
        hq = (item - b * packs) * p.pack_heads;       // first head of the pack
    } else {
        const int per_group = p.n_q_tiles * p.heads_per_group;
        const int group = item / per_group;
        const int bh0 = group * p.heads_per_group;
        const int group_size = (n_bh - bh0 < p.heads_per_group) ? (n_bh - bh0) : p.heads_per_group;
        const int local = item - group * per_group;
        q_tile = p.n_q_tiles - 1 - local / group_size;
        const int bh = bh0 + local % group_size;
        hq = bh % p.Hq;
        b = bh / p.Hq;
    }
    const int kvh = hq / (p.Hq / p.Hkv);
    int Sq = p.Sq, Sk = p.Sk, q_row0 = 0, k_row0 = 0;
    if constexpr (kVarlen) {
        q_row0 = p.cu_q[b];
        k_row0 = p.cu_k[b];
        Sq = p.cu_q[b + 1] - q_row0;
        Sk = p.cu_k[b + 1] - k_row0;
    }
    const int off = Sk - Sq;
    const int i0 = q_tile * kTileM;
    if (kVarlen && i0 >= Sq) return;      // a sequence shorter than the longest one (whole CTA, before any set-up)
    // K/V tiles [j_base, j_base + n_kv) of the query tile belong to this CTA (all visible ones without split-KV)
    // (packed batches: the host does not know the lengths, so the C equal shares are cut here)
    const int n_kv_all = kv_tiles_for_q_tile(i0, kTileM, Sq, Sk, p.causal);
    const int tiles_per_split = (kVarlen && p.kv_splits > 1) ? (n_kv_all + p.kv_splits - 1) / p.kv_splits : p.tiles_per_split;
    const int j_base = split * tiles_per_split;
    int n_kv = n_kv_all - j_base;
    if (n_kv > tiles_per_split) n_kv = tiles_per_split;
    if (n_kv < 0) n_kv = 0;
    const int tb = kVarlen ? 0 : b;       // batch coordinate of the tensor maps (packed tensors have one slice)

    // ---------------------------------------------------------------- setup
    if (tid == 0) {
        sh.abort_flag = 0;
        mbar_init(smem_addr(&sh.q_full), 1);
        mbar_init(smem_addr(&sh.o_final), 1);
        mbar_init(smem_addr(&sh.l_ready), 8);
        mbar_init(smem_addr(&sh.o_staged), 8);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_addr(&sh.s_full[i]), 1);
            mbar_init(smem_addr(&sh.s_free[i]), 4);       // the 4 warps of warpgroup i
            mbar_init(smem_addr(&sh.st_full[i]), 4);
            mbar_init(smem_addr(&sh.p_ready[i]), 8);      // 4 softmax warps + 4 correction warps
            mbar_init(smem_addr(&sh.p_free[i]), 1);
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
    if constexpr (kPack) {
        // the rows of the query tile past the pack's last row are never loaded: zero scores there
        for (int o = tid * 16; o < Cfg::kQBytes; o += 512 * 16) st_shared_v4(sQ + o, 0u, 0u, 0u, 0u);
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if constexpr (!kVarlen) grid_dependency_wait();

    const uint32_t tmem_base = sh.tmem_base;
    WaitCtx wctx{&sh.abort_flag, p.status, p.wait_limit_ns};
    const float c = p.scale_log2;

    if (warp < 8) {
        // ============================================================ softmax of K/V tiles j = g, g+2, ...
        setmaxnreg_inc<kRegsSoftmax>();
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
        // the query this thread's row belongs to: index in its sequence, head, and whether it exists
        // (packed batches: every head's rows are p.Sq apart in the tile, the longest query of the
        // batch, and a shorter sequence leaves the rest of its head's rows unused)
        const int pack_rows = kVarlen ? p.Sq : Sq;
        const int h_local = kPack ? row / pack_rows : 0;
        const int i_glob = kPack ? row - h_local * pack_rows : i0 + row;
        const bool row_valid = kPack ? (h_local < p.pack_heads && i_glob < Sq) : (i_glob < Sq);
        const int hq_row = hq + h_local;
        const int q_idx = b * p.Hq + hq_row;
        int kmax_row = Sk - 1;
        if (p.causal && i_glob + off < kmax_row) kmax_row = i_glob + off;
        const float tau_raw = kRescaleThresholdLog2 / c;

        float l = 0.f;             // this warpgroup's partial row sum, relative to the current u
        bool ok = true;
        for (int j = g; j < n_kv; j += 2) {
            const uint32_t use = static_cast<uint32_t>(j >> 1);       // n-th use of this warpgroup's buffers
            ok = __all_sync(0xffffffffu, mbar_wait(bar_s, use & 1u, wctx, kSiteSoftmaxSFull));
            if (!ok) break;
            tc_fence_after_sync();
            const int j0 = (j_base + j) * kTileN;
            const bool need_mask = (j0 + kTileN - 1 > kmax_row);

            uint32_t s[kTileN];
            tmem_ld_x32(tS + 0, s + 0);
            tmem_ld_x32(tS + 32, s + 32);
            tmem_ld_x32(tS + 64, s + 64);
            tmem_ld_x32(tS + 96, s + 96);
            tc_wait_ld();
            // S^g is in registers: the score MMA of tile j+2 may overwrite it
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

            // Row state of tile j-1 from the other warpgroup: u, and the factor r it applied.
            float m_ref = -INFINITY, r_prev = 1.f;
            if (j > 0) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar_st_other, static_cast<uint32_t>((j - 1) >> 1) & 1u, wctx,
                                                       kSiteSoftmaxCorrFree));
                if (!ok) break;
                m_ref = sh.mref[row];
                r_prev = sh.alpha[(j - 1) & 1][row];
            }
            // P^g and the slot of this tile's r are reused every second tile: the PV MMA of tile j-2
            // must be complete.  It was issued a whole tile ago, so this wait is normally over at
            // once; it also means that the correction warps have consumed r of tile j-2, which
            // keeps the next phase of st_full from overtaking them (a parity wait cannot tell a
            // phase from the one two phases later).
            if (j >= 2) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar_pf, (use - 1u) & 1u, wctx, kSiteSoftmaxPFree));
                if (!ok) break;
            }
            float alpha = 1.f;
            if (mx > m_ref + tau_raw) {
                alpha = exp2_approx((m_ref - mx) * c);    // r = exp(u' - u); 0 on the first tile
                m_ref = mx;
            }
            sh.mref[row] = m_ref;
            sh.alpha[j & 1][row] = alpha;
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
            // conversion and store of a chunk run under the exponentials of the next one
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

        // ---- epilogue: O = G' / s (bf16), lse = u * scale + ln s
        if (ok && i0 < Sq) {
            // fixed lengths: lse [B, Hq, Sq]; packed batches: lse [Hq, total_q], O rows q_row0 onwards
            const size_t lse_row0 = kVarlen ? static_cast<size_t>(hq_row) * p.total_q + q_row0 : static_cast<size_t>(q_idx) * p.Sq;
            const long long o_base = (kVarlen ? q_row0 * p.o_stride_s : b * p.o_stride_b) + hq_row * p.o_stride_h;
            if (p.kv_splits > 1 && n_kv == 0) {      // an empty range: a neutral partial
                if (row_valid) {
                    const size_t prow = kVarlen ? (static_cast<size_t>(split) * p.Hq + hq_row) * p.total_q + q_row0 + i_glob
                                                : (static_cast<size_t>(split) * n_bh + q_idx) * p.Sq + i_glob;
                    float* po_row = p.o_part + prow * DV + g * (DV / 2);
                    const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int v = 0; v < DV / 8; ++v) reinterpret_cast<float4*>(po_row)[v] = z;
                    if (g == 0) p.lse_part[prow] = -INFINITY;
                }
            } else if (n_kv == 0) {       // no key visible to any row of this tile
                if (g == 0 && row_valid) {
                    __nv_bfloat16* o_row = p.O + (o_base + static_cast<long long>(i_glob) * p.o_stride_s);
                    const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int v = 0; v < DV / 8; ++v) reinterpret_cast<uint4*>(o_row)[v] = z;
                    if (p.lse) p.lse[lse_row0 + i_glob] = -INFINITY;
                }
            } else {
                // The warpgroup that did not run the last tile still has to apply its r.
                const int last = n_kv - 1;
                if ((last & 1) != g && last >= 1) {
                    // st_full of the last tile: also orders the read of alpha and mref below
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_st_other, static_cast<uint32_t>(last >> 1) & 1u, wctx,
                                                           kSiteSoftmaxCorrFree));
                    if (ok) l *= sh.alpha[last & 1][row];
                }
                if (ok) {
                    sh.lsum[g][row] = (g <= last) ? l : 0.f;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_addr(&sh.l_ready));
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.l_ready), 0, wctx, kSiteEpiStaged));
                }
                if (ok) ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.o_final), 0, wctx, kSiteEpiOFull));
                if (ok) {
                    tc_fence_after_sync();
                    const float lt = sh.lsum[0][row] + sh.lsum[1][row];
                    const float m_fin = sh.mref[row];
                    const float inv_l = (lt > 0.f) ? (1.f / lt) : 0.f;
                    if (g == 0 && p.lse && row_valid && p.kv_splits == 1)
                        p.lse[lse_row0 + i_glob] = (lt > 0.f) ? (m_fin * c * 0.6931471805599453f + logf(lt)) : -INFINITY;
                    // warpgroup g converts columns [g*DV/2, (g+1)*DV/2) of O into the staging tile
                    // (the Q tile's space: the last score MMA is long complete), then one thread
                    // stores it with TMA; rows past Sq are clipped
                    const uint32_t tO = tmem_base + Cfg::kColO + lane_sel;
                    // the last tile of a packed sequence is followed by the next sequence's rows, which a
                    // box store would overwrite: it is stored row by row
                    const bool box_store = !kVarlen || (i0 + kTileM <= Sq);
                    if (p.kv_splits > 1) {
                        // split-KV: G'_c / s_c in fp32 and u_c + ln s_c go to scratch (Algorithm 2's partials)
                        // fixed lengths: partials [C, B*Hq, Sq]; packed batches: [C, Hq, total_q]
                        const size_t prow = kVarlen ? (static_cast<size_t>(split) * p.Hq + hq_row) * p.total_q + q_row0 + i_glob
                                                    : (static_cast<size_t>(split) * n_bh + q_idx) * p.Sq + i_glob;
                        float* po_row = p.o_part + prow * DV;
                        if (g == 0 && row_valid)
                            p.lse_part[prow] = (lt > 0.f) ? (m_fin * c * 0.6931471805599453f + logf(lt)) : -INFINITY;
#pragma unroll 1
                        for (int cc = g * (DV / 64); cc < (g + 1) * (DV / 64); ++cc) {
                            uint32_t r[32];
                            tmem_ld_x32(tO + cc * 32, r);
                            tc_wait_ld();
                            if (row_valid) {
#pragma unroll
                                for (int v = 0; v < 8; ++v)
                                    reinterpret_cast<float4*>(po_row + cc * 32)[v] = make_float4(
                                        __uint_as_float(r[4 * v]) * inv_l, __uint_as_float(r[4 * v + 1]) * inv_l,
                                        __uint_as_float(r[4 * v + 2]) * inv_l, __uint_as_float(r[4 * v + 3]) * inv_l);
                            }
                        }
                    } else if (box_store) {
                        const uint32_t sO = sQ + row * 128;
#pragma unroll 1
                        for (int cc = g * (DV / 64); cc < (g + 1) * (DV / 64); ++cc) {
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
                        if (lane == 0) mbar_arrive(smem_addr(&sh.o_staged));
                        if (warp == 0 && lane == 0 && mbar_wait(smem_addr(&sh.o_staged), 0, wctx, kSiteEpiStaged)) {
#pragma unroll
                            for (int ch = 0; ch < DV / kChunkCols; ++ch)
                                tma_store_4d(&tm_o, sQ + ch * kChunkBytes, ch * kChunkCols, q_row0 + i0, hq, tb);
                            tma_store_commit();
                            tma_store_wait_read_all();     // the CTA's shared memory outlives the reads
                        }
                    } else {
                        __nv_bfloat16* o_row = p.O + (o_base + static_cast<long long>(i_glob) * p.o_stride_s);
#pragma unroll 1
                        for (int cc = g * (DV / 64); cc < (g + 1) * (DV / 64); ++cc) {
                            uint32_t r[32];
                            tmem_ld_x32(tO + cc * 32, r);
                            tc_wait_ld();
                            if (row_valid) {
#pragma unroll
                                for (int v = 0; v < 4; ++v)
                                    reinterpret_cast<uint4*>(o_row + cc * 32)[v] = make_uint4(
                                        pack_bf16x2(__uint_as_float(r[8 * v]) * inv_l, __uint_as_float(r[8 * v + 1]) * inv_l),
                                        pack_bf16x2(__uint_as_float(r[8 * v + 2]) * inv_l, __uint_as_float(r[8 * v + 3]) * inv_l),
                                        pack_bf16x2(__uint_as_float(r[8 * v + 4]) * inv_l, __uint_as_float(r[8 * v + 5]) * inv_l),
                                        pack_bf16x2(__uint_as_float(r[8 * v + 6]) * inv_l, __uint_as_float(r[8 * v + 7]) * inv_l));
                            }
                        }
                    }
                }
            }
        }
    } else if (warp < 12) {
        // ============================================================ correction of the O accumulator
        setmaxnreg_dec<kRegsCorrection>();
        const int row = tid & (kTileM - 1);
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tO = tmem_base + Cfg::kColO + lane_sel;
        bool ok = true;
        for (int j = 0; j < n_kv && ok; ++j) {
            const uint32_t use = static_cast<uint32_t>(j >> 1);
            ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.st_full[j & 1]), use & 1u, wctx, kSiteCorrScale));
            if (!ok) break;
            const float alpha = sh.alpha[j & 1][row];
            if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                // O must hold the complete sum up to tile j-1 before it is rescaled
                ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.p_free[(j - 1) & 1]),
                                                       static_cast<uint32_t>((j - 1) >> 1) & 1u, wctx, kSiteCorrPvDone));
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
            if (lane == 0) mbar_arrive(smem_addr(&sh.p_ready[j & 1]));
        }
    } else if (warp == 12) {
        // ============================================================ score MMAs: S^(j&1) = Q K_j^T
        setmaxnreg_dec<kRegsOther>();
        if (elect_one() && n_kv > 0) {
            constexpr uint32_t kIdescQK = make_idesc_bf16_f32(kTileM, kTileN, false, false);
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // sbo, version, swizzle
            const uint32_t q_lo = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
            auto desc = [](uint32_t lo) -> uint64_t { return (static_cast<uint64_t>(kDescHi) << 32) | lo; };
            bool ok = mbar_wait(smem_addr(&sh.q_full), 0, wctx, kSiteMmaQFull);
            int sk = 0;
            uint32_t ph_k = 0;
            for (int j = 0; j < n_kv && ok; ++j) {
                const uint32_t use = static_cast<uint32_t>(j >> 1);
                ok = mbar_wait(smem_addr(&sh.k_full[sk]), ph_k, wctx, kSiteMmaKvFull);
                if (ok && j >= 2) ok = mbar_wait(smem_addr(&sh.s_free[j & 1]), (use - 1u) & 1u, wctx, kSiteMmaSFree);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t tS = tmem_base + Cfg::kColS + (j & 1) * 128;
                const uint32_t klo = k_lo0 + sk * (Cfg::kKBytes >> 4);
#pragma unroll
                for (int k = 0; k < DQK / 16; ++k) {
                    const uint32_t koff = ((k / 4) * kChunkBytes + (k % 4) * 32) >> 4;
                    mma_ss(tS, desc(q_lo + koff), desc(klo + koff), kIdescQK, k > 0 ? 1u : 0u);
                }
                tc_commit(smem_addr(&sh.s_full[j & 1]));
                tc_commit(smem_addr(&sh.k_empty[sk]));
                if (++sk == NK) { sk = 0; ph_k ^= 1u; }
            }
        }
    } else if (warp == 13) {
        // ============================================================ PV MMAs: O += P^(j&1) V_j
        setmaxnreg_dec<kRegsOther>();
        if (elect_one() && n_kv > 0) {
            constexpr uint32_t kIdescPV = make_idesc_bf16_f32(kTileM, DV, false, true);
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
            const uint32_t v_lo0 = ((sV & 0x3FFFFu) >> 4) | ((static_cast<uint32_t>(kChunkBytes) >> 4) << 16);
            const uint32_t tO = tmem_base + Cfg::kColO;
            auto desc = [](uint32_t lo) -> uint64_t { return (static_cast<uint64_t>(kDescHi) << 32) | lo; };
            int sv = 0;
            uint32_t ph_v = 0;
            bool ok = true;
            for (int j = 0; j < n_kv && ok; ++j) {
                const uint32_t use = static_cast<uint32_t>(j >> 1);
                ok = mbar_wait(smem_addr(&sh.v_full[sv]), ph_v, wctx, kSiteMmaKvFull);
                if (ok) ok = mbar_wait(smem_addr(&sh.p_ready[j & 1]), use & 1u, wctx, kSiteMmaPFull);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t tP = tmem_base + Cfg::kColP + (j & 1) * 64;
                const uint32_t vlo = v_lo0 + sv * (Cfg::kVBytes >> 4);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ts(tO, tP + kk * 8, desc(vlo + kk * (2048 >> 4)), kIdescPV, (j > 0 || kk > 0) ? 1u : 0u);
                tc_commit(smem_addr(&sh.p_free[j & 1]));
                tc_commit(smem_addr(&sh.v_empty[sv]));
                if (j + 1 == n_kv) tc_commit(smem_addr(&sh.o_final));
                if (++sv == NV) { sv = 0; ph_v ^= 1u; }
            }
        }
    } else if (warp == 14) {
        // ============================================================ TMA loads of Q and K
        // K and V have a loading thread each: a V stage is only free again after the PV MMA that
        // runs behind a whole softmax, and one thread loading both in turn would hold the K loads
        // (which the score MMAs want two tiles ahead) back behind it.
        setmaxnreg_dec<kRegsOther>();
        if (elect_one() && n_kv > 0) {
            {
                const uint32_t bar = smem_addr(&sh.q_full);
                // with packed heads the box is Sq rows x pack_heads heads (row h * Sq + i of the tile)
                mbar_arrive_expect_tx(bar, kPack ? static_cast<uint32_t>(Cfg::kQChunks * p.pack_heads * (kVarlen ? p.Sq : Sq) * 128)
                                                 : static_cast<uint32_t>(Cfg::kQBytes));
#pragma unroll
                for (int cc = 0; cc < Cfg::kQChunks; ++cc)
                    tma_load_4d(sQ + cc * kChunkBytes, &tm_q, bar, cc * kChunkCols, q_row0 + i0, hq, tb);
            }
            bool ok = true;
            for (int j = 0; j < n_kv && ok; ++j) {
                const int s = j % NK;
                ok = mbar_wait(smem_addr(&sh.k_empty[s]), ((j / NK) & 1) ^ 1, wctx, kSiteLoadKvEmpty);
                if (!ok) break;
                const uint32_t bar = smem_addr(&sh.k_full[s]);
                mbar_arrive_expect_tx(bar, Cfg::kKBytes);
#pragma unroll
                for (int cc = 0; cc < Cfg::kQChunks; ++cc)
                    tma_load_4d(sK + s * Cfg::kKBytes + cc * kChunkBytes, &tm_k, bar, cc * kChunkCols, k_row0 + (j_base + j) * kTileN, kvh, tb);
            }
        }
    } else {
        // ============================================================ warp 15: TMA loads of V
        setmaxnreg_dec<kRegsOther>();
        if (elect_one() && n_kv > 0) {
            bool ok = true;
            for (int j = 0; j < n_kv && ok; ++j) {
                if (p.debug_drop_v_load && j == 0) continue;      // (test hook: see FA_FLAG_DEBUG_DROP_V_LOAD)
                const int s = j % NV;
                ok = mbar_wait(smem_addr(&sh.v_empty[s]), ((j / NV) & 1) ^ 1, wctx, kSiteLoadKvEmpty);
                if (!ok) break;
                const uint32_t bar = smem_addr(&sh.v_full[s]);
                mbar_arrive_expect_tx(bar, Cfg::kVBytes);
#pragma unroll
                for (int cc = 0; cc < Cfg::kVChunks; ++cc)
                    tma_load_4d(sV + s * Cfg::kVBytes + cc * kChunkBytes, &tm_v, bar, cc * kChunkCols, k_row0 + (j_base + j) * kTileN, kvh, tb);
            }
        }
    }

    // ---------------------------------------------------------------- teardown (all warps)
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 12) tmem_dealloc(tmem_base, Cfg::kTmemCols);
}

}  // namespace fa
