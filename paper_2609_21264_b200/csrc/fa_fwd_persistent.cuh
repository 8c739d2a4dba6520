// Persistent variant of the pipelined attention forward kernel for sm_100a.
//
// Same roles, same arithmetic and the same per-round schedule as fa_fwd_pipelined.cuh (read that
// file first), but a CTA does not end with its pair of query tiles: the grid is one CTA per SM
// and every CTA walks a static list of work items (item = pair of adjacent query tiles of one
// (batch, head)), so that
//   * the set-up (barriers, TMEM, tensor-map fetch) and the launch of a new CTA are paid once per
//     SM instead of once per item,
//   * the loads of the next item (Q as soon as the last score MMA of a tile is done, K/V as soon
//     as a ring stage is free) and its first score MMA run under the tail of the current item,
//   * the final normalisation of a tile goes through a staging buffer of its own and a TMA
//     store, so only the TMEM read-out of O_t (a few hundred cycles) sits between the last
//     P_t V of one item and the first softmax of the next.
// It pays off when items are short (a CTA's fixed cost is then a large share of its time) and
// there are more items than SMs; the host picks it for those launches only.
//
// Items are ordered longest first (as in the non-persistent grid).  CTA c starts with item c;
// every further item is drawn from a global ticket counter by the K/V load thread once the loads
// of the current item are all issued, decoded by that thread (the divisions of the decode take a
// lone thread over a thousand cycles) and handed to the other roles through a four-slot ring in
// shared memory, so a CTA that got short items simply takes more of them.  Every CTA draws
// exactly one ticket past the end of the list, which makes the total number of draws known: the
// CTA that takes the last one puts the counter back to zero for the next launch.  All mbarrier
// phases, ring stages and the strict alternation of the two MMA-issuing threads run on across
// items.
//
// Differences in the roles: warp 15 (idle in the non-persistent kernel) loads the Q tiles, warp
// 14 only K and V; two K stages instead of three at d = 128 make room for the staging buffer.
// No split-KV.  kVarlen = packed variable-length batch: an item's lengths and row offsets are read
// from p.cu_q / p.cu_k when it is decoded; the list has an item for every tile (pair) of the
// longest sequence, and the items a shorter sequence does not have pass through the ring empty.
#pragma once

#include "fa_fwd_pipelined.cuh"

namespace fa {

template <int DQK, int DV>
struct PersistCfg {
    using Base = PipeCfg<DQK, DV>;
    static constexpr int kQBytes = Base::kQBytes;
    static constexpr int kKBytes = Base::kKBytes;
    static constexpr int kVBytes = Base::kVBytes;
    static constexpr int kOBytes = (DV / kChunkCols) * kChunkBytes;     // one bf16 output tile
    static constexpr int kKStages = (DQK == 128) ? 2 : 4;
    static constexpr int kVStages = (DQK == 128) ? 2 : 4;
    static constexpr int kTileBytes = 2 * kQBytes + kKStages * kKBytes + kVStages * kVBytes + kOBytes;
};

// One work item, decoded from its place in the longest-first order.
struct alignas(16) PersistItem {
    int b, hq, kvh;
    int Sq, Sk;              // lengths of the item's sequence (the launch's, or the packed sequence's)
    int q_row0, k_row0;      // first rows of the sequence in the packed tensors (0 with fixed lengths)
    int hq1;                 // query head of tile 1 (the same head, or the next one when heads are paired)
    int i0_0, i0_1;          // first rows of the two query tiles (128 rows apart, or equal when heads are paired)
    int nkv_0, nkv_1, n_max; // K/V tiles of tile 0, tile 1, and the larger of the two
    int pad[3];
};
static_assert(sizeof(PersistItem) == 64, "the item ring moves items as four 16-byte words");

struct PersistShared {
    uint64_t q_full[2];      // Q loader -> MMA thread t: Q_t of the item is in shared memory
    uint64_t q_empty[2];     // MMA thread t -> Q loader: last score MMA of the item has read Q_t
    uint64_t k_full[4], k_empty[4];
    uint64_t v_full[4], v_empty[4];
    uint64_t s_full[2];      // MMA -> softmax: S_t(j) is in TMEM
    uint64_t p_half[2];      // softmax + correction -> MMA: keys 0..63 of P_t(j) written, O_t rescaled
    uint64_t p_full[2];      // softmax -> MMA: all of P_t(j) written
    uint64_t scale_full[2];  // softmax -> correction: alpha of iteration j published
    uint64_t o_final[2];     // MMA -> softmax: last PV of tile t done, O_t is final
    uint64_t turn[2];        // MMA thread 1-t -> MMA thread t: your turn to issue
    uint64_t stage_full;     // softmax warps -> storing thread: the bf16 O tile is in the staging buffer
    uint64_t stage_empty;    // storing thread -> softmax warps: the TMA store has read the staging buffer
    uint64_t item_full[4];   // K/V load thread -> every role: item_ring[slot] holds the next work item
    uint64_t item_empty[4];  // every role -> K/V load thread: slot read (8 + 4 warps, 2 MMA threads, Q loader)
    int item_ring[4];        // index of the item in the list (>= the list's length: the end mark)
    PersistItem items[4];    // the item itself, decoded once by the K/V load thread
    float alpha[2][2][kTileM];   // [tile][iteration & 1][row]
    uint32_t tmem_base;
    uint32_t abort_flag;
};

template <int DQK, int DV>
constexpr int persist_smem_bytes() {
    return PersistCfg<DQK, DV>::kTileBytes + static_cast<int>(sizeof(PersistShared));
}

template <bool kVarlen = false>
__device__ __forceinline__ PersistItem persist_decode(const FwdParams& p, int idx) {
    // Groups of (batch, head) instances whose K/V fit in L2 together follow one another; inside a
    // group every head's last (with a causal mask: heaviest) pair comes first.
    // With paired heads (p.head_pair) an item is ONE query tile of two adjacent query heads of a
    // K/V group, as in the pair kernel's kHeadPair mode, and the units below are pairs of heads.
    const int hp = p.head_pair;
    const int n_pairs = hp ? p.n_q_tiles : (p.n_q_tiles + 1) / 2;
    const int n_units = hp ? p.B * p.Hq / 2 : p.B * p.Hq;
    const int hpg = hp ? p.heads_per_group / 2 : p.heads_per_group;
    const int per_group = n_pairs * hpg;
    const int group = idx / per_group;
    const int bh0 = group * hpg;
    const int group_size = (n_units - bh0 < hpg) ? (n_units - bh0) : hpg;
    const int local = idx - group * per_group;
    const int pair = n_pairs - 1 - local / group_size;
    const int bh = hp ? 2 * (bh0 + local % group_size) : bh0 + local % group_size;
    PersistItem it;
    it.hq = bh % p.Hq;
    it.hq1 = it.hq + hp;
    it.b = bh / p.Hq;
    it.kvh = it.hq / (p.Hq / p.Hkv);
    it.i0_0 = (hp ? pair : 2 * pair) * kTileM;
    it.i0_1 = hp ? it.i0_0 : it.i0_0 + kTileM;
    it.Sq = p.Sq; it.Sk = p.Sk; it.q_row0 = 0; it.k_row0 = 0;
    if constexpr (kVarlen) {
        it.q_row0 = p.cu_q[it.b];
        it.k_row0 = p.cu_k[it.b];
        it.Sq = p.cu_q[it.b + 1] - it.q_row0;
        it.Sk = p.cu_k[it.b + 1] - it.k_row0;
    }
    it.nkv_0 = (it.i0_0 < it.Sq) ? kv_tiles_for_q_tile(it.i0_0, kTileM, it.Sq, it.Sk, p.causal) : 0;
    it.nkv_1 = (it.i0_1 < it.Sq) ? kv_tiles_for_q_tile(it.i0_1, kTileM, it.Sq, it.Sk, p.causal) : 0;
    it.n_max = it.nkv_0 > it.nkv_1 ? it.nkv_0 : it.nkv_1;
    return it;
}

template <int DQK, int DV, bool kVarlen = false>
__global__ void __launch_bounds__(512, 1)
fa_fwd_persistent_kernel(const __grid_constant__ CUtensorMap tm_q,
                         const __grid_constant__ CUtensorMap tm_k,
                         const __grid_constant__ CUtensorMap tm_v,
                         const __grid_constant__ CUtensorMap tm_o,
                         const FwdParams p) {
    using Cfg = PersistCfg<DQK, DV>;
    using Base = PipeCfg<DQK, DV>;
    using namespace ptx;
    constexpr int NK = Cfg::kKStages;
    constexpr int NV = Cfg::kVStages;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    PersistShared& sh = *reinterpret_cast<PersistShared*>(smem_raw + Cfg::kTileBytes);

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
            mbar_init(smem_addr(&sh.p_half[t]), 8);       // 4 softmax warps + 4 correction warps
            mbar_init(smem_addr(&sh.p_full[t]), 4);       // 4 softmax warps
            mbar_init(smem_addr(&sh.scale_full[t]), 4);
            mbar_init(smem_addr(&sh.o_final[t]), 1);
            mbar_init(smem_addr(&sh.turn[t]), 1);
        }
        mbar_init(smem_addr(&sh.stage_full), 4);          // 4 softmax warps of the tile being stored
        mbar_init(smem_addr(&sh.stage_empty), 1);
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            mbar_init(smem_addr(&sh.item_full[s]), 1);
            mbar_init(smem_addr(&sh.item_empty[s]), 15);
            mbar_init(smem_addr(&sh.k_full[s]), 1);
            mbar_init(smem_addr(&sh.k_empty[s]), 2);      // one arrival per MMA-issuing thread
            mbar_init(smem_addr(&sh.v_full[s]), 1);
            mbar_init(smem_addr(&sh.v_empty[s]), 2);
        }
        fence_mbar_init();
    }
    if (warp == 12) {
        tmem_alloc(smem_addr(&sh.tmem_base), Base::kTmemCols);
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

    // Consumer side of the work-item ring: the k-th item of this CTA, or -1 at the end of the list
    // (or when a wait gave up).  The warp form is called by all lanes of a warp together.
    // A consumer waits for slot k & 3, copies what it needs (item_at) and releases the slot; the softmax
    // warps, which need the item again in their epilogue, release it at the end of the item instead.
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
        setmaxnreg_inc<kRegsSoftmax>();
        const int t = warp >> 2;
        const int row = tid & (kTileM - 1);
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + (t == 0 ? Base::kColS0 : Base::kColS1) + lane_sel;
        const uint32_t tO = tmem_base + (t == 0 ? Base::kColO0 : Base::kColO1) + lane_sel;
        const uint32_t bar_s = smem_addr(&sh.s_full[t]);
        const uint32_t bar_p = smem_addr(&sh.p_full[t]);
        const uint32_t bar_ph = smem_addr(&sh.p_half[t]);
        const uint32_t bar_scale = smem_addr(&sh.scale_full[t]);
        const float tau_raw = kRescaleThresholdLog2 / c;
        uint32_t it = 0;       // iterations of this tile so far, over all items: barrier parities
        uint32_t oc = 0;       // items with work for this tile so far: parity of o_final
        uint32_t uc = 0;       // uses of the staging buffer so far, by either tile
        bool ok = true;

#pragma unroll 1
        for (int k = 0; ok; item_release(k), ++k) {      // (the slot is kept until the item's epilogue has read it again)
            if (item_wait(k) < 0) break;
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
                tc_fence_after_sync();
                const int j0 = j * kTileN;
                const bool need_mask = (j0 + kTileN - 1 > kmax_row);

                const float2 c2 = make_float2(c, c);
                float2 nmc2;
                float2 sum_a = make_float2(0.f, 0.f), sum_b = make_float2(0.f, 0.f);
                float alpha = 1.f;
                uint32_t s[kTileN];
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
                    tmem_st_x16(tS + q * 16, pk);
                };
                // speculative exponentials against the carried-over reference maximum; see the
                // non-persistent kernel
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
                sh.alpha[t][it & 1u][row] = alpha;
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
            if (!ok) break;

            // ---- epilogue of the item: O = G' / s (bf16), lse = u * scale + ln s
            if (i0_t >= Sq) continue;
            const PersistItem item = item_at(k);     // again: nothing of it was kept live
            const int hq_t = t == 0 ? item.hq : item.hq1;
            // fixed lengths: lse [B, Hq, Sq]; packed batches: lse [Hq, total_q], O rows q_row0 onwards
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
            tc_fence_after_sync();
            const float inv_l = (l > 0.f) ? (1.f / l) : 0.f;
            if (p.lse && i_glob < Sq)
                p.lse[lse_row0 + i_glob] = (l > 0.f) ? (m_ref * c * 0.6931471805599453f + logf(l)) : -INFINITY;
            // A packed batch's last tile of a sequence is followed by the next sequence's rows, which a
            // box store would overwrite: every warp copies the rows it staged to global memory itself
            // (one 256-byte bulk copy per row out of the staging buffer measured 5-15 % slower).
            const bool box_store = !kVarlen || (i0_t + kTileM <= Sq);
            // the previous user's TMA store must have read the staging buffer
            ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.stage_empty), (my_use & 1u) ^ 1u, wctx, kSiteEpiStaged));
            if (!ok) break;
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
        }
        // all bulk stores of this thread have left shared memory (waited for above); their global
        // writes are complete when the grid is
    } else if (warp < 12) {
        // ============================================================ correction of the O accumulators
        setmaxnreg_dec<kRegsCorrection>();
        const int row = tid & (kTileM - 1);
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        uint32_t it0 = 0, it1 = 0;
        bool ok = true;
#pragma unroll 1
        for (int k = 0; ok; ++k) {
            if (item_wait(k) < 0) break;
            const PersistItem item = item_at(k);
            item_release(k);
#pragma unroll 1
            for (int j = 0; j < item.n_max && ok; ++j) {
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (j >= (t == 0 ? item.nkv_0 : item.nkv_1) || !ok) continue;
                    const uint32_t itt = (t == 0) ? it0 : it1;
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_addr(&sh.scale_full[t]), itt & 1u, wctx,
                                                           kSiteCorrScale));
                    if (!ok) break;
                    const float alpha = sh.alpha[t][itt & 1u][row];
                    if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                        tc_fence_after_sync();
                        const uint32_t tO = tmem_base + (t == 0 ? Base::kColO0 : Base::kColO1) + lane_sel;
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
                    if (t == 0) ++it0; else ++it1;
                }
            }
        }
    } else if (warp == 12 || warp == 13) {
        // ============================================================ MMA issue for tile t = warp - 12
        setmaxnreg_dec<kRegsOther>();
        if (elect_one()) {
            const int t = warp - 12;
            constexpr uint32_t kIdescQK = make_idesc_bf16_f32(kTileM, kTileN, false, false);
            constexpr uint32_t kIdescPV = make_idesc_bf16_f32(kTileM, DV, false, true);
            constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // sbo, version, swizzle
            const uint32_t q_lo = (((sQ + t * Cfg::kQBytes) & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t k_lo0 = ((sK & 0x3FFFFu) >> 4) | (1u << 16);
            const uint32_t v_lo0 = ((sV & 0x3FFFFu) >> 4) | ((static_cast<uint32_t>(kChunkBytes) >> 4) << 16);
            const uint32_t tS = tmem_base + (t == 0 ? Base::kColS0 : Base::kColS1);   // P_t overlays it
            const uint32_t tO = tmem_base + (t == 0 ? Base::kColO0 : Base::kColO1);
            const uint32_t bar_s = smem_addr(&sh.s_full[t]);
            const uint32_t bar_ph = smem_addr(&sh.p_half[t]);
            const uint32_t bar_p = smem_addr(&sh.p_full[t]);
            const uint32_t bar_qe = smem_addr(&sh.q_empty[t]);
            auto desc = [](uint32_t lo) -> uint64_t {
                return (static_cast<uint64_t>(kDescHi) << 32) | lo;
            };
            auto issue_qk = [&](int stage) {
                const uint32_t klo = k_lo0 + stage * (Cfg::kKBytes >> 4);
#pragma unroll
                for (int kk = 0; kk < DQK / 16; ++kk) {
                    const uint32_t koff = ((kk / 4) * kChunkBytes + (kk % 4) * 32) >> 4;
                    mma_ss(tS, desc(q_lo + koff), desc(klo + koff), kIdescQK, kk > 0 ? 1u : 0u);
                }
            };
            auto issue_pv_half = [&](auto hc, int stage, uint32_t accumulate) {
                constexpr int half = decltype(hc)::value;
                const uint32_t vlo = v_lo0 + stage * (Cfg::kVBytes >> 4);
#pragma unroll
                for (int kk = 4 * half; kk < 4 * half + 4; ++kk)
                    mma_ts(tO, tS + kk * 8, desc(vlo + kk * (2048 >> 4)), kIdescPV,
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

            int sk = 0, sv = 0;                  // stage of the next K tile and the next V tile to consume
            uint32_t ph_k = 0, ph_v = 0;
            uint32_t it = 0;                     // iterations with work for this tile so far
            uint32_t qc = 0;                     // items with work for this tile so far (parity of q_full)
            bool ok = true;
#pragma unroll 1
            for (int k = 0; ok; ++k) {
                if (item_wait_thread(k) < 0) break;
                int nkv_t, n_max;
                {
                    const PersistItem item = item_at(k);
                    nkv_t = (t == 0) ? item.nkv_0 : item.nkv_1;
                    n_max = item.n_max;
                }
                item_release_thread(k);
                if (n_max == 0) continue;
                // First block of the item: S_t(0) = Q_t K_0^T.  It is issued as soon as its operands
                // are there, outside the alternation of the two threads: the other thread may still
                // be in the last round of the previous item, and waiting for it would put this
                // tile's whole chain on hold.
                ok = mbar_wait(smem_addr(&sh.k_full[sk]), ph_k, wctx, kSiteMmaKvFull);
                if (ok && nkv_t > 0) { ok = mbar_wait(smem_addr(&sh.q_full[t]), qc & 1u, wctx, kSiteMmaQFull); ++qc; }
                if (!ok) break;
                if (nkv_t > 0) {
                    tc_fence_after_sync();
                    issue_qk(sk);
                    tc_commit(bar_s);
                    if (nkv_t == 1) tc_commit(bar_qe);      // that was the last score MMA of the item
                }
                tc_commit(smem_addr(&sh.k_empty[sk]));
                if (++sk == NK) { sk = 0; ph_k ^= 1u; }
#pragma unroll 1
                for (int j = 0; j < n_max; ++j) {
                    // Both threads wait for every stage, also on iterations without work for their
                    // tile, so that neither arrives twice in one phase of an "empty" barrier.
                    ok = mbar_wait(smem_addr(&sh.v_full[sv]), ph_v, wctx, kSiteMmaKvFull);
                    if (ok && j + 1 < n_max) ok = mbar_wait(smem_addr(&sh.k_full[sk]), ph_k, wctx, kSiteMmaKvFull);
                    if (ok && j < nkv_t) ok = mbar_wait(bar_ph, it & 1u, wctx, kSiteMmaPFull);
                    ok = ok && take_turn();
                    if (!ok) break;
                    tc_fence_after_sync();
                    if (j < nkv_t) {
                        issue_pv_half(IntC<0>{}, sv, j > 0 ? 1u : 0u);
                        ok = mbar_wait(bar_p, it & 1u, wctx, kSiteMmaPFull);
                        if (!ok) break;
                        tc_fence_after_sync();
                        issue_pv_half(IntC<1>{}, sv, 1u);
                        ++it;
                    }
                    if (j + 1 < nkv_t) {
                        issue_qk(sk);
                        tc_commit(bar_s);
                        if (j + 2 == nkv_t) tc_commit(bar_qe);  // last score MMA of the item: Q_t may be replaced
                    } else if (j + 1 == nkv_t) {
                        tc_commit(smem_addr(&sh.o_final[t]));
                    }
                    tc_commit(smem_addr(&sh.v_empty[sv]));
                    if (++sv == NV) { sv = 0; ph_v ^= 1u; }
                    if (j + 1 < n_max) {
                        tc_commit(smem_addr(&sh.k_empty[sk]));
                        if (++sk == NK) { sk = 0; ph_k ^= 1u; }
                    }
                    pass_turn();
                }
            }
        }
    } else if (warp == 14) {
        // ============================================================ TMA loads of K and V
        setmaxnreg_dec<kRegsOther>();
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
                        for (int cc = 0; cc < Base::kQChunks; ++cc)
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
                        for (int cc = 0; cc < Base::kVChunks; ++cc)
                            tma_load_4d(sV + s * Cfg::kVBytes + cc * kChunkBytes, &tm_v, bar, cc * kChunkCols,
                                        item.k_row0 + j0, item.kvh, kVarlen ? 0 : item.b);
                        ++vc;
                    }
                }
                // Draw the next item only now that the loads of this one are all issued (the rings
                // keep this thread a tile or two ahead of the MMAs): an earlier draw would bind an
                // item to this CTA long before it can start on it (starting the atomic ahead of the
                // loads of short items, to hide its round trip, measured 1-4 % slower).  The launch
                // makes n_items draws in all (n_items - G that return an item, one past the end per CTA).
                const unsigned int ticket = atomicAdd(p.sched_counter, 1u);
                if (ticket == static_cast<unsigned int>(n_items) - 1u) atomicExch(p.sched_counter, 0u);
                idx = G + static_cast<int>(ticket);
            }
        }
    } else {
        // ============================================================ warp 15: TMA loads of the Q tiles
        setmaxnreg_dec<kRegsOther>();
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
                    for (int cc = 0; cc < Base::kQChunks; ++cc)
                        tma_load_4d(sQ + t * Cfg::kQBytes + cc * kChunkBytes, &tm_q, bar, cc * kChunkCols,
                                    item.q_row0 + (t == 0 ? item.i0_0 : item.i0_1), t == 0 ? item.hq : item.hq1,
                                    kVarlen ? 0 : item.b);
                    if (t == 0) ++qc0; else ++qc1;
                }
            }
        }
    }

    // ---------------------------------------------------------------- teardown (all warps)
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 12) tmem_dealloc(tmem_base, Base::kTmemCols);
}

}  // namespace fa
