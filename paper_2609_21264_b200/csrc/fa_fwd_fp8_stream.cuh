// Block-scaled e4m3 attention forward, one 128-row query tile per CTA with its K/V tiles streamed
// through both softmax warpgroups: the 8-bit operand format of fa_fwd_fp8.cuh (Q and K with one
// fp32 scale per 128-row tile, V with one per head, P rounded to e4m3, both contractions on
// tcgen05.mma kind::f8f6f4) on the tiling and protocol of fa_fwd_stream.cuh.  Read those two
// files first; nothing else is new here.  The block scales of Q and K multiply a whole score
// tile and are folded into the exp2 constant of that tile, so the reference maximum that the
// two warpgroups hand to each other is kept in scaled log2 units.  Used by fa_forward_fp8 where
// the stream tiling is planned: grids under a wave and decode-like shapes with split-KV
// (attention over an 8-bit K/V cache).  Head sizes 64, 128 and 192/128, fixed-length contiguous tensors.
//   TMEM  S^0 [0,128)  S^1 [128,256)  O [256,384)  P^0 [384,416)  P^1 [448,480)
//
// kMx: the MX form of the operands (the closest counterpart of a block floating point format on this GPU): e4m3
// codes with one e8m0 scale per 32 elements ALONG THE CONTRACTION, for Q and K per row and block of the head
// dimension, for V per column and block of 32 keys, applied inside tcgen05.mma kind::mxf8f6f4.block_scale.
// Nothing is folded into the exp2 constant then.  The scales of a 128-row tile arrive as one 512-byte atom next
// to the tile (a plain bulk copy on the tile's mbarrier) and go from shared memory to TMEM columns
// [416,440) with tcgen05.cp, issued by the MMA thread that uses them, just ahead of the tile's MMAs; P is
// rounded to e4m3 as before and carries the scale 1 (one constant atom).
//   TMEM  scales: Q [416,420)  K^0 [420,424)  K^1 [424,428)  P [428,432)  V^0 [432,436)  V^1 [436,440)
#pragma once

#include "fa_fwd_fp8.cuh"
#include "fa_fwd_stream.cuh"

namespace fa {

// D = head size of Q and K; V and O have the same, except D = 192, where they have 128 (the 192/128 shapes).
// A Q or K row of 192 bytes is two swizzled chunks: columns [0,128) with the 128-byte swizzle (16 KB per
// 128-row tile) and columns [128,192) with the 64-byte swizzle (8 KB), each with a tensor map of its own.
template <int D>
struct Fp8StreamCfg {
    static_assert(D == 64 || D == 128 || D == 192, "head sizes of the 8-bit stream kernel");
    static constexpr int kD = D;
    static constexpr int kDV = (D == 192) ? 128 : D;
    static constexpr int kTile8 = kTileM * kD;           // one 128 x D e4m3 tile of Q or K (8, 16 or 24 KB)
    static constexpr int kVTile8 = kTileM * kDV;         // one 128 x DV e4m3 tile of V
    static constexpr int kOBytes = (kDV / kChunkCols) * kChunkBytes;      // bf16 output tile
    static constexpr int kKStages = 4;
    static constexpr int kVStages = 4;
    static constexpr int kSfAtom = 512;                  // scales of one 128-row tile (MX variant)
    static constexpr int kSfBytes = (2 + kKStages + kVStages) * kSfAtom;     // Q, P (constant), K and V stages
    static constexpr int kTileBytes = (1 + kKStages) * kTile8 + kVStages * kVTile8 + kOBytes + kSfBytes;
    static constexpr int kTmemCols = 512;
    static constexpr int kColS = 0, kColO = 256, kColP = 384;   // P^b at kColP + 64 b (32 columns used)
    static constexpr int kColSf = 416;
    // shared-memory descriptor high words (stride between 8-row groups, version, swizzle mode) of a chunk with
    // 128-byte and with 64-byte rows
    static constexpr uint32_t kDescHi128 = (1024u >> 4) | (1u << 14) | (2u << 29);
    static constexpr uint32_t kDescHi64 = (512u >> 4) | (1u << 14) | (4u << 29);
    static constexpr uint32_t kDescHiQK = (D == 64) ? kDescHi64 : kDescHi128;      // first chunk of Q and K
    static constexpr uint32_t kDescHiV = (kDV == 64) ? kDescHi64 : kDescHi128;
    static constexpr uint32_t kVStep = (32u * kDV) >> 4;  // 32 keys of V, in descriptor address units
};

template <int D>
constexpr int fp8_stream_smem_bytes() { return Fp8StreamCfg<D>::kTileBytes + static_cast<int>(sizeof(StreamShared)); }

// kPack: several query heads of one K/V head share the query tile, as in fa_fwd_stream_kernel.
// kRep (with kPack, 2 or 4): the pack has at most 128 / kRep rows and is loaded kRep times, copy
// r into rows [r * 128 / kRep, (r + 1) * 128 / kRep) of the query tile.  Copy r only takes the
// keys [r * 128 / kRep, ...) of every K/V tile: its threads read that slice of the score tile,
// exponentiate it and write that slice of P, whose other columns stay zero.  The copies are thus
// kRep independent attention problems over disjoint keys, each with its own row state, and they
// leave the kernel as kRep partials per split, merged by fa_combine_kernel like split-KV
// partials.  A softmax warp then issues 1 / kRep of the exponentials per K/V tile (an
// instruction costs the same for one live row as for 32), which takes a few-row problem from the
// MUFU bound to the bound of the K/V stream.
template <int D, bool kPack = false, int kRep = 1, bool kMx = false>
__global__ void __launch_bounds__(512, 1)
fa_fwd_fp8_stream_kernel(const __grid_constant__ CUtensorMap tm_q,
                     const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v,
                     const __grid_constant__ CUtensorMap tm_o,
                     const __grid_constant__ CUtensorMap tm_q2,    // D = 192: columns [128,192) of Q and of K
                     const __grid_constant__ CUtensorMap tm_k2,    // (64-byte swizzle); otherwise unused
                     const FwdParams p, const Fp8Params f) {
    using Cfg = Fp8StreamCfg<D>;
    constexpr int DV = Cfg::kDV;
    constexpr int kTile8 = Cfg::kTile8;
    constexpr int kVTile8 = Cfg::kVTile8;
    static_assert(D != 192 || (!kPack && !kMx), "192/128: one head per query tile, fp32 block scales");
    static_assert(kRep == 1 || (kPack && (kRep == 2 || kRep == 4)), "copies of the query rows need packed heads");
    static_assert(!kMx || !kPack, "the MX variant has no packed heads (its scale atoms follow the query tile's rows)");
    constexpr int kRepRows = kTileM / kRep;      // rows of one copy of the pack
    constexpr int kCols = kTileN / kRep;         // keys of a K/V tile that one copy takes
    constexpr int kChunks = kCols / 32;
    using namespace ptx;
    constexpr int NK = Cfg::kKStages;
    constexpr int NV = Cfg::kVStages;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    StreamShared& sh = *reinterpret_cast<StreamShared*>(smem_raw + Cfg::kTileBytes);

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
    const uint32_t sK = sQ + kTile8;
    const uint32_t sV = sK + NK * kTile8;
    const uint32_t sStage = sV + NV * kVTile8;     // the bf16 output tile passes through here
    const uint32_t sSfQ = sStage + Cfg::kOBytes;   // scale atoms (MX variant): Q, P, K stages, V stages
    const uint32_t sSfP = sSfQ + Cfg::kSfAtom;
    const uint32_t sSfK = sSfP + Cfg::kSfAtom;
    const uint32_t sSfV = sSfK + NK * Cfg::kSfAtom;

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
    const int kv_idx = b * p.Hkv + kvh;
    const int Sq = p.Sq, Sk = p.Sk;
    const int off = Sk - Sq;
    const int i0 = q_tile * kTileM;
    // K/V tiles [j_base, j_base + n_kv) of the query tile belong to this CTA (all visible ones without split-KV)
    const int j_base = split * p.tiles_per_split;
    int n_kv = kv_tiles_for_q_tile(i0, kTileM, Sq, Sk, p.causal) - j_base;
    if (n_kv > p.tiles_per_split) n_kv = p.tiles_per_split;
    if (n_kv < 0) n_kv = 0;

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
    if constexpr (kMx) {
        // P carries the scale 1 = 2^(127 - 127) in every block
        if (tid < Cfg::kSfAtom / 16) st_shared_v4(sSfP + tid * 16, 0x7f7f7f7fu, 0x7f7f7f7fu, 0x7f7f7f7fu, 0x7f7f7f7fu);
        fence_proxy_async_smem();
    }
    if constexpr (kPack) {
        // the rows of the query tile past the pack's last row are never loaded: zero scores there
        for (int o = tid * 16; o < kTile8; o += 512 * 16) st_shared_v4(sQ + o, 0u, 0u, 0u, 0u);
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    grid_dependency_wait();

    const uint32_t tmem_base = sh.tmem_base;
    WaitCtx wctx{&sh.abort_flag, p.status, p.wait_limit_ns};

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
        const int copy = row / kRepRows;              // which copy of the pack (0 without copies)
        const int row_in_copy = row - copy * kRepRows;
        const int h_local = kPack ? row_in_copy / Sq : 0;
        const int i_glob = kPack ? row_in_copy - h_local * Sq : i0 + row;
        const int col0 = copy * kCols;                // first key of a tile that this row takes
        const bool partial_out = p.kv_splits > 1 || kRep > 1;
        const int part = split * kRep + copy;         // index of this row's partial
        const bool row_valid = kPack ? (h_local < p.pack_heads) : (i_glob < Sq);
        const int hq_row = hq + h_local;
        const int q_idx = b * p.Hq + hq_row;
        int kmax_row = Sk - 1;
        if (p.causal && i_glob + off < kmax_row) kmax_row = i_glob + off;
        // scale * log2 e * (scale of this query tile); the key tile's scale joins per tile
        // (MX variant: the scales are applied inside the MMAs)
        const float cq = p.scale_log2 * ((!kMx && f.q_scale && row_valid) ? __ldg(f.q_scale + static_cast<size_t>(q_idx) * p.n_q_tiles + q_tile) : 1.f);
        const float* k_scale = (!kMx && f.k_scale) ? f.k_scale + static_cast<size_t>(kv_idx) * f.n_kv_tiles + j_base : nullptr;

        if constexpr (kRep > 1) {
            // the columns of P^g that belong to the other copies' keys are never written: zero once
            uint32_t z[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) z[e] = 0u;
            tmem_st_x32(tP, z);
            tc_wait_st();
        }
        float l = 0.f;             // this warpgroup's partial row sum, relative to the current u
        bool ok = true;
        for (int j = g; j < n_kv; j += 2) {
            const uint32_t use = static_cast<uint32_t>(j >> 1);       // n-th use of this warpgroup's buffers
            const float c = cq * (k_scale ? __ldg(k_scale + j) : 1.f);  // exp2 argument = raw score * c - u
            ok = __all_sync(0xffffffffu, mbar_wait(bar_s, use & 1u, wctx, kSiteSoftmaxSFull));
            if (!ok) break;
            tc_fence_after_sync();
            const int j0 = (j_base + j) * kTileN;
            const bool need_mask = (j0 + kTileN - 1 > kmax_row);

            uint32_t s[kCols];
#pragma unroll
            for (int q = 0; q < kChunks; ++q) tmem_ld_x32(tS + col0 + q * 32, s + q * 32);
            tc_wait_ld();
            // S^g is in registers: the score MMA of tile j+2 may overwrite it
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_sf);
            if (need_mask) {
#pragma unroll
                for (int e = 0; e < kCols; ++e)
                    if (j0 + col0 + e > kmax_row) s[e] = 0xff800000u;   // -inf
            }
            float a[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) a[q] = -INFINITY;
#pragma unroll
            for (int e = 0; e < kCols; e += 16) {
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    a[q] = fmax3(a[q], __uint_as_float(s[e + 2 * q]), __uint_as_float(s[e + 2 * q + 1]));
            }
            float mx = fmaxf(fmax3(a[0], a[1], a[2]), fmax3(a[3], a[4], a[5]));
            mx = fmax3(mx, a[6], a[7]) * c;     // scaled log2 units (c > 0: the maximum commutes with the scaling)

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
            if (mx > m_ref + kRescaleThresholdLog2) {
                alpha = exp2_approx(m_ref - mx);          // r = exp(u' - u); 0 on the first tile
                m_ref = mx;
            }
            sh.mref[row] = m_ref;
            sh.alpha[j & 1][row] = alpha;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_st);

            const float mc = (m_ref == -INFINITY) ? 0.f : m_ref;
            const float2 c2 = make_float2(c, c);
            const float2 nmc2 = make_float2(-mc, -mc);
            float2 sum_a = make_float2(0.f, 0.f), sum_b = make_float2(0.f, 0.f);
            auto exp_chunk = [&](int q) {
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[q * 32 + e]),
                                                            __uint_as_float(s[q * 32 + e + 1])), c2, nmc2);
                    // (every kFp8EmuEvery-th pair on the FMA pipe: the 8-bit loop is MUFU-bound, see fa_fwd_fp8.cuh)
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
                tmem_st_x8(tP + col0 / 4 + q * 8, pk);
            };
            // conversion and store of a chunk run under the exponentials of the next one
            exp_chunk(0);
#pragma unroll
            for (int q = 1; q < kChunks; ++q) {
                exp_chunk(q);
                emit_chunk(q - 1);
            }
            emit_chunk(kChunks - 1);
            l = l * (r_prev * alpha) + ((sum_a.x + sum_a.y) + (sum_b.x + sum_b.y));
            tc_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_pr);
        }

        // ---- epilogue: O = G' / s (bf16), lse = u * scale + ln s
        if (ok && i0 < Sq) {
            const size_t lse_row0 = static_cast<size_t>(q_idx) * p.Sq;
            const long long o_base = b * p.o_stride_b + hq_row * p.o_stride_h;
            if (partial_out && n_kv == 0) {      // an empty range: a neutral partial
                if (row_valid) {
                    const size_t prow = (static_cast<size_t>(part) * n_bh + q_idx) * p.Sq + i_glob;
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
                    const float sv = (!kMx && f.v_scale) ? __ldg(f.v_scale + kv_idx) : 1.f;
                    const float inv_l = (lt > 0.f) ? (sv / lt) : 0.f;
                    if (g == 0 && p.lse && row_valid && !partial_out)
                        p.lse[lse_row0 + i_glob] = (lt > 0.f) ? (m_fin * 0.6931471805599453f + logf(lt)) : -INFINITY;
                    // warpgroup g converts columns [g*DV/2, (g+1)*DV/2) of O into the staging tile
                    // (the Q tile's space: the last score MMA is long complete), then one thread
                    // stores it with TMA; rows past Sq are clipped
                    const uint32_t tO = tmem_base + Cfg::kColO + lane_sel;
                    if (partial_out) {
                        // split-KV: G'_c / s_c in fp32 and u_c + ln s_c go to scratch (Algorithm 2's partials)
                        const size_t prow = (static_cast<size_t>(part) * n_bh + q_idx) * p.Sq + i_glob;
                        float* po_row = p.o_part + prow * DV;
                        if (g == 0 && row_valid)
                            p.lse_part[prow] = (lt > 0.f) ? (m_fin * 0.6931471805599453f + logf(lt)) : -INFINITY;
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
                    } else {
                        const uint32_t sO = sStage + row * 128;
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
                                tma_store_4d(&tm_o, sStage + ch * kChunkBytes, ch * kChunkCols, i0, hq, b);
                            tma_store_commit();
                            tma_store_wait_read_all();     // the CTA's shared memory outlives the reads
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
            constexpr uint32_t kIdescQK = make_idesc_e4m3_f32(kTileM, kTileN, false, false);
            constexpr uint32_t kDescHi = Cfg::kDescHiQK;
            const uint32_t q_lo = ((sQ & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
            auto desc = [](uint32_t lo) -> uint64_t { return (static_cast<uint64_t>(kDescHi) << 32) | lo; };
            auto desc64 = [](uint32_t lo) -> uint64_t { return (static_cast<uint64_t>(Cfg::kDescHi64) << 32) | lo; };
            bool ok = mbar_wait(smem_addr(&sh.q_full), 0, wctx, kSiteMmaQFull);
            if constexpr (kMx) {
                if (ok) {
                    tc_fence_after_sync();
                    tmem_cp_scales_32x16B(tmem_base + Cfg::kColSf, sSfQ);
                }
            }
            int sk = 0;
            uint32_t ph_k = 0;
            for (int j = 0; j < n_kv && ok; ++j) {
                const uint32_t use = static_cast<uint32_t>(j >> 1);
                ok = mbar_wait(smem_addr(&sh.k_full[sk]), ph_k, wctx, kSiteMmaKvFull);
                if (ok && j >= 2) ok = mbar_wait(smem_addr(&sh.s_free[j & 1]), (use - 1u) & 1u, wctx, kSiteMmaSFree);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t tS = tmem_base + Cfg::kColS + (j & 1) * 128;
                const uint32_t klo = k_lo0 + sk * (kTile8 >> 4);
                if constexpr (kMx) {
                    const uint32_t tSfK = tmem_base + Cfg::kColSf + 4 + (j & 1) * 4;
                    tmem_cp_scales_32x16B(tSfK, sSfK + sk * Cfg::kSfAtom);
#pragma unroll
                    for (int kk = 0; kk < Cfg::kD / 32; ++kk)      // K block kk of Q's rows and of K's rows
                        mma_ss_mx(tS, desc(q_lo + kk * 2), desc(klo + kk * 2), make_idesc_mx_e4m3(kTileM, kTileN, false, kk, kk),
                                  tmem_base + Cfg::kColSf, tSfK, kk > 0 ? 1u : 0u);
                } else {
#pragma unroll
                    for (int kk = 0; kk < (D == 192 ? 4 : Cfg::kD / 32); ++kk)      // k-steps of 32 elements = 32 bytes
                        mma_ss_f8(tS, desc(q_lo + kk * 2), desc(klo + kk * 2), kIdescQK, kk > 0 ? 1u : 0u);
                    if constexpr (D == 192) {
                        // columns [128,192): the second chunk of Q and of K (64-byte rows), 16 KB behind the first
#pragma unroll
                        for (int kk = 0; kk < 2; ++kk)
                            mma_ss_f8(tS, desc64(q_lo + (16384 >> 4) + kk * 2), desc64(klo + (16384 >> 4) + kk * 2), kIdescQK, 1u);
                    }
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
            constexpr uint32_t kIdescPV = make_idesc_e4m3_f32(kTileM, DV, false, true);
            constexpr uint32_t kDescHi = Cfg::kDescHiV;
            const uint32_t v_lo0 = ((sV & 0x3FFFFu) >> 4) | ((16384u >> 4) << 16);   // one swizzled row spans dv: the chunk stride is not used
            const uint32_t tO = tmem_base + Cfg::kColO;
            auto desc = [](uint32_t lo) -> uint64_t { return (static_cast<uint64_t>(kDescHi) << 32) | lo; };
            int sv = 0;
            uint32_t ph_v = 0;
            bool ok = true;
            if constexpr (kMx) tmem_cp_scales_32x16B(tmem_base + Cfg::kColSf + 12, sSfP);     // (written before the set-up barrier)
            for (int j = 0; j < n_kv && ok; ++j) {
                const uint32_t use = static_cast<uint32_t>(j >> 1);
                ok = mbar_wait(smem_addr(&sh.v_full[sv]), ph_v, wctx, kSiteMmaKvFull);
                if (ok) ok = mbar_wait(smem_addr(&sh.p_ready[j & 1]), use & 1u, wctx, kSiteMmaPFull);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t tP = tmem_base + Cfg::kColP + (j & 1) * 64;
                const uint32_t vlo = v_lo0 + sv * (kVTile8 >> 4);
                if constexpr (kMx) {
                    const uint32_t tSfV = tmem_base + Cfg::kColSf + 16 + (j & 1) * 4;
                    tmem_cp_scales_32x16B(tSfV, sSfV + sv * Cfg::kSfAtom);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)              // block kk of the tile's keys: P's scale (1) and V's per column
                        mma_ts_mx(tO, tP + kk * 8, desc(vlo + kk * Cfg::kVStep), make_idesc_mx_e4m3(kTileM, DV, true, kk, kk),
                                  tmem_base + Cfg::kColSf + 12, tSfV, (j > 0 || kk > 0) ? 1u : 0u);
                } else {
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)              // four k-steps of 32 keys: 8 P columns, 32 V rows of D bytes
                        mma_ts_f8(tO, tP + kk * 8, desc(vlo + kk * Cfg::kVStep), kIdescPV, (j > 0 || kk > 0) ? 1u : 0u);
                }
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
                mbar_arrive_expect_tx(bar, (kPack ? static_cast<uint32_t>(kRep * p.pack_heads * Sq * D) : static_cast<uint32_t>(kTile8)) +
                                               (kMx ? Cfg::kSfAtom : 0));
#pragma unroll
                for (int r = 0; r < kRep; ++r) tma_load_4d(sQ + r * kRepRows * D, &tm_q, bar, 0, i0, hq, b);
                if constexpr (D == 192) tma_load_4d(sQ + 16384, &tm_q2, bar, 128, i0, hq, b);
                if constexpr (kMx)
                    bulk_load_1d(sSfQ, f.q_sf + (static_cast<size_t>(b * p.Hq + hq) * p.n_q_tiles + q_tile) * Cfg::kSfAtom, Cfg::kSfAtom, bar);
            }
            bool ok = true;
            for (int j = 0; j < n_kv && ok; ++j) {
                const int s = j % NK;
                ok = mbar_wait(smem_addr(&sh.k_empty[s]), ((j / NK) & 1) ^ 1, wctx, kSiteLoadKvEmpty);
                if (!ok) break;
                const uint32_t bar = smem_addr(&sh.k_full[s]);
                mbar_arrive_expect_tx(bar, kTile8 + (kMx ? Cfg::kSfAtom : 0));
                tma_load_4d(sK + s * kTile8, &tm_k, bar, 0, (j_base + j) * kTileN, kvh, b);
                if constexpr (D == 192) tma_load_4d(sK + s * kTile8 + 16384, &tm_k2, bar, 128, (j_base + j) * kTileN, kvh, b);
                if constexpr (kMx)
                    bulk_load_1d(sSfK + s * Cfg::kSfAtom, f.k_sf + (static_cast<size_t>(kv_idx) * f.n_kv_tiles + j_base + j) * Cfg::kSfAtom,
                                 Cfg::kSfAtom, bar);
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
                mbar_arrive_expect_tx(bar, kVTile8 + (kMx ? Cfg::kSfAtom : 0));
                tma_load_4d(sV + s * kVTile8, &tm_v, bar, 0, (j_base + j) * kTileN, kvh, b);
                if constexpr (kMx)
                    bulk_load_1d(sSfV + s * Cfg::kSfAtom, f.v_sf + (static_cast<size_t>(kv_idx) * f.n_kv_tiles + j_base + j) * Cfg::kSfAtom,
                                 Cfg::kSfAtom, bar);
            }
        }
    }

    // ---------------------------------------------------------------- teardown (all warps)
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 12) tmem_dealloc(tmem_base, Cfg::kTmemCols);
}

}  // namespace fa
