// The softmax pass of the kernels built on the loop of fa_fwd_pair.cuh (fa_fwd_pair_kernel, its persistent form
// and the two-CTA kernel): one thread owns one query row of a 128 x 128 score tile in TMEM.
//
// Online softmax of Algorithm 1 for one K/V tile, with the state kept in fp32 and the scale folded into the
// exponent: scores S -> P = 2^((S - u) c) as bf16 over the first half of S, running row sum l, lazily advanced
// reference maximum u (m_ref, raw score units; it only moves when a row maximum exceeds it by more than
// kRescaleThresholdLog2 in log2 units, so P stays below 2^8).
//   * The first 32 exponentials are issued against the carried reference maximum while the row maximum of the
//     tile is still being reduced; if any row of the warp needs a new reference the pass is repeated from TMEM
//     (nothing has been stored yet, S is intact).
//   * On the rare tiles where a reference moved, the warp multiplies its own 32 rows of the O accumulator by
//     r = 2^((u_old - u_new) c) in TMEM before it hands P over: the PV product of the previous tile of this
//     accumulator is complete (S could not be visible otherwise) and the next one waits for the hand-off.
//   * P is handed over in two parts, keys 0..95 (arrive_first) and 96..127 (arrive_rest), each after
//     tcgen05.wait::st and tcgen05.fence::before_thread_sync, by lane 0 of the warp.
//   * The row sum is taken after the hand-off, off the chain MMA -> softmax -> MMA.
#pragma once

#include <math.h>

#include "fa_common.cuh"
#include "ptx.cuh"

namespace fa {

// tS: TMEM address of this warp's lanes of the score tile (P overlays its first 64 columns); tO: of the accumulator
// that P_t V_j goes to; c = scale * log2(e); tau_raw = kRescaleThresholdLog2 / c; keys j0 + e > kmax_row are masked;
// first_tile: nothing has been accumulated into O yet (no rescale).  All 32 lanes of a warp call it together.
template <int DV, typename ArriveFirst, typename ArriveRest>
FA_DEVI void softmax_pass_128(uint32_t tS, uint32_t tO, float c, float tau_raw, int j0, int kmax_row, bool first_tile,
                              float& m_ref, float& l, int lane, ArriveFirst&& arrive_first, ArriveRest&& arrive_rest) {
    using namespace ptx;
    const bool need_mask = (j0 + kTileN - 1 > kmax_row);
    const float2 c2 = make_float2(c, c);
    float2 nmc2;
    float2 sum_a = make_float2(0.f, 0.f), sum_b = make_float2(0.f, 0.f);
    float alpha = 1.f;
    uint32_t s[kTileN];
    auto exp_chunk = [&](int q) {
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
            const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[q * 32 + e]), __uint_as_float(s[q * 32 + e + 1])), c2, nmc2);
            s[q * 32 + e] = __float_as_uint(exp2_approx(x.x));
            s[q * 32 + e + 1] = __float_as_uint(exp2_approx(x.y));
        }
    };
    // bf16 conversion and store of one chunk of P (over the first half of S)
    auto emit_chunk = [&](int q) {
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 32; e += 2)
            pk[e / 2] = pack_bf16x2(__uint_as_float(s[q * 32 + e]), __uint_as_float(s[q * 32 + e + 1]));
        tmem_st_x16(tS + q * 16, pk);
    };
    auto sum_chunk = [&](int q) {
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
            sum_a = fadd2_ftz(sum_a, make_float2(__uint_as_float(s[q * 32 + e]), __uint_as_float(s[q * 32 + e + 1])));
            sum_b = fadd2_ftz(sum_b, make_float2(__uint_as_float(s[q * 32 + e + 2]), __uint_as_float(s[q * 32 + e + 3])));
        }
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
    if (!first_tile && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll 1
        for (int cc = 0; cc < DV / 32; ++cc) {
            uint32_t r[32];
            tmem_ld_x32(tO + cc * 32, r);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e)
                r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
            tmem_st_x32(tO + cc * 32, reinterpret_cast<uint32_t(&)[32]>(r));
        }
    }
    exp_chunk(1);
    emit_chunk(0);
    exp_chunk(2);
    emit_chunk(1);
    emit_chunk(2);
    // keys 0..95 of P are stored: the MMA thread may start O += P V on them
    tc_wait_st();
    tc_fence_before_sync();
    __syncwarp();
    if (lane == 0) arrive_first();
    exp_chunk(3);
    emit_chunk(3);
    tc_wait_st();
    tc_fence_before_sync();
    __syncwarp();
    if (lane == 0) arrive_rest();
    sum_chunk(0);
    sum_chunk(1);
    sum_chunk(2);
    sum_chunk(3);
    l = l * alpha + ((sum_a.x + sum_a.y) + (sum_b.x + sum_b.y));
}

}  // namespace fa
