// Inline-PTX wrappers for sm_100a: mbarrier (bounded waits), TMA tensor loads,
// tcgen05 (TMEM allocation, MMA, commit, ld/st, fences) and descriptor builders.
// Everything here is device-only and header-only; no library code is used.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#define FA_DEVI __device__ __forceinline__

namespace fa {
namespace ptx {

// ------------------------------------------------------------------ misc

FA_DEVI uint32_t smem_addr(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

FA_DEVI uint64_t globaltimer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

FA_DEVI bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "elect.sync _|p, 0xffffffff;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(pred));
    return pred != 0;
}

FA_DEVI float exp2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// exp2 of two values on the FMA pipe instead of the MUFU: the integer part n = floor(x) is taken with the
// 1.5 * 2^23 trick (an addition rounded towards minus infinity leaves n in the low mantissa bits), the fraction
// f = x - n in [0, 1) goes through a cubic (minimax fit of 2^f, relative error 7.5e-5, far below the rounding of P
// to bf16 or e4m3 that follows), and n is put back with a shift and an integer add into the exponent field.
// Valid for x < 127.  x below -125 (masked scores are -inf) is clamped there and comes out as about 2^-125, which
// rounds to zero in P and vanishes in the row sum; the clamp must stay above -126, where the integer add would
// carry out of the exponent field and produce a NaN pattern.
FA_DEVI float2 exp2_poly2(float2 x) {
    const float kMagic = 12582912.f;
    x.x = fmaxf(x.x, -125.f);
    x.y = fmaxf(x.y, -125.f);
    unsigned long long xb, yb, mb;
    asm("mov.b64 %0, {%1, %2};" : "=l"(xb) : "f"(x.x), "f"(x.y));
    asm("mov.b64 %0, {%1, %1};" : "=l"(mb) : "f"(kMagic));
    asm("add.rm.ftz.f32x2 %0, %1, %2;" : "=l"(yb) : "l"(xb), "l"(mb));
    float2 y;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(y.x), "=f"(y.y) : "l"(yb));
    const float2 nf = __fadd2_rn(y, make_float2(-kMagic, -kMagic));
    const float2 f = __fadd2_rn(x, make_float2(-nf.x, -nf.y));
    float2 p = __ffma2_rn(make_float2(7.8024521470e-02f, 7.8024521470e-02f), f, make_float2(2.2606717050e-01f, 2.2606717050e-01f));
    p = __ffma2_rn(p, f, make_float2(6.9583350420e-01f, 6.9583350420e-01f));
    p = __ffma2_rn(p, f, make_float2(9.9992519617e-01f, 9.9992519617e-01f));
    float2 r;
    r.x = __uint_as_float(__float_as_uint(p.x) + (__float_as_uint(y.x) << 23));
    r.y = __uint_as_float(__float_as_uint(p.y) + (__float_as_uint(y.y) << 23));
    return r;
}

// a + b on two lanes, denormal inputs and results flushed to zero
FA_DEVI float2 fadd2_ftz(float2 a, float2 b) {
    unsigned long long ab, bb, rb;
    asm("mov.b64 %0, {%1, %2};" : "=l"(ab) : "f"(a.x), "f"(a.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(bb) : "f"(b.x), "f"(b.y));
    asm("add.rn.ftz.f32x2 %0, %1, %2;" : "=l"(rb) : "l"(ab), "l"(bb));
    float2 r;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(r.x), "=f"(r.y) : "l"(rb));
    return r;
}

FA_DEVI float fmax3(float a, float b, float c) {
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}

// Two fp32 -> packed bf16x2 (lo in bits [0,16), hi in bits [16,32)), round to nearest even.
FA_DEVI uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Four fp32 -> packed e4m3x4 (f0 in bits [0,8) ... f3 in bits [24,32)), round to nearest even,
// saturating to the largest finite value.
FA_DEVI uint32_t pack_e4m3x4(float f0, float f1, float f2, float f3) {
    uint16_t lo, hi;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(f1), "f"(f0));
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(f3), "f"(f2));
    uint32_t r;
    asm("mov.b32 %0, {%1, %2};" : "=r"(r) : "h"(lo), "h"(hi));
    return r;
}

template <int kRegs>
FA_DEVI void setmaxnreg_inc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegs));
}
template <int kRegs>
FA_DEVI void setmaxnreg_dec() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegs));
}

FA_DEVI void named_barrier_sync(uint32_t id, uint32_t nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// ------------------------------------------------------------------ mbarrier

FA_DEVI void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
FA_DEVI void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// Makes generic-proxy writes to shared memory visible to the async proxy (TMA, tcgen05).
FA_DEVI void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
FA_DEVI void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
FA_DEVI void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
FA_DEVI bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Shared between all roles of a CTA: once any wait gives up, every other wait
// returns false promptly so that all roles fall through to the common exit.
struct WaitCtx {
    volatile uint32_t* abort_flag;   // in shared memory
    uint32_t* status;                // global (mapped host) status words, may be NULL
    uint64_t limit_ns;
};

// Bounded wait on an mbarrier phase.  Returns false if the wait ran out (or if
// another role already gave up); then records `who` in the status word.
FA_DEVI bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx& ctx, uint32_t who) {
    if (mbar_try_wait(bar, parity)) return true;
    uint64_t t0 = 0;
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (*ctx.abort_flag) return false;
            const uint64_t now = globaltimer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > ctx.limit_ns) {
                *ctx.abort_flag = 1u;
                if (ctx.status) {
                    volatile uint32_t* sw = ctx.status;   // mapped host memory: plain stores
                    sw[1] = who;
                    sw[0] = 4u;                           // FA_ERR_DEVICE_TIMEOUT
                    __threadfence_system();
                }
                return false;
            }
        }
    }
}

// ------------------------------------------------------------------ programmatic dependent launch

// Lets the next kernel of the stream (if it was launched with programmatic stream serialisation)
// be scheduled as soon as every CTA of this grid has got here or has exited.
FA_DEVI void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// Blocks until the preceding kernel of the stream has completed and its writes are visible.  A
// no-op for a kernel that was launched the ordinary way.  Must come before the first access to
// global memory that an earlier kernel may have written, and every CTA must pass it before it
// exits (a grid whose CTAs skipped it could finish before its predecessor, and its own successor,
// which waits for this grid only, would then overtake that predecessor).
FA_DEVI void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ------------------------------------------------------------------ TMA

FA_DEVI void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// 3-D tiled load global -> shared, completion on an mbarrier (bytes).  The
// innermost coordinate c0 must keep c0 * elemsize a multiple of 16 bytes.
FA_DEVI void tma_load_3d(uint32_t dst_smem, const CUtensorMap* map, uint32_t bar,
                         int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar),
          "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// 4-D tiled load global -> shared (coordinates: column, row, head, batch).
FA_DEVI void tma_load_4d(uint32_t dst_smem, const CUtensorMap* map, uint32_t bar,
                         int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar),
          "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}

// 3-D tiled store shared -> global (bulk async group).
FA_DEVI void tma_store_3d(const CUtensorMap* map, uint32_t src_smem, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
        ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src_smem), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
// 4-D tiled store shared -> global (coordinates: column, row, head, batch); rows and columns of
// the box that fall outside the tensor are not written.
FA_DEVI void tma_store_4d(const CUtensorMap* map, uint32_t src_smem, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
        ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src_smem), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
FA_DEVI void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
FA_DEVI uint4 ld_shared_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
// A warp's 32 rows of a bf16 output tile, staged in the swizzled layout of a TMA box (64-column
// chunks of 128 rows x 128 bytes, 16-byte pieces XORed with the row's low three bits), go to global
// memory coalesced: consecutive lanes take consecutive 16-byte pieces of a row, so one instruction
// covers whole rows instead of 32 rows' pieces.  Rows from `valid_rows` on are skipped.  For the
// tiles that cannot leave as one TMA box (the last, partly filled tile of a packed sequence).
// tile_smem: the tile's staging area; row0: the warp's first row in it; tile_global: address of
// the tile's row 0, column 0; stride: elements between rows.  The caller has synchronised the warp
// after its own stores into the staging area (every lane staged row0 + lane).
template <int DV>
FA_DEVI void store_staged_rows(uint32_t tile_smem, int row0, int valid_rows, __nv_bfloat16* tile_global,
                               long long stride, int lane) {
    constexpr int kPieces = DV / 8;                  // 16-byte pieces per row
    constexpr int kRowsPerPass = 32 / kPieces;
    const int piece = lane % kPieces;
#pragma unroll 4
    for (int rr = 0; rr < 32; rr += kRowsPerPass) {
        const int r = row0 + rr + lane / kPieces;
        const uint4 v = ld_shared_v4(tile_smem + (piece >> 3) * (128 * 128) + r * 128 + (((piece & 7) ^ (r & 7)) << 4));
        if (r < valid_rows) *reinterpret_cast<uint4*>(tile_global + r * stride + piece * 8) = v;
    }
}
FA_DEVI void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
FA_DEVI void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
FA_DEVI void tma_store_wait_read_all() {
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// ------------------------------------------------------------------ tcgen05: TMEM management

// One full warp executes these (.sync.aligned).  ncols: power of two in [32, 512].
FA_DEVI void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_dst), "r"(ncols) : "memory");
}
FA_DEVI void tmem_relinquish_alloc_permit() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
FA_DEVI void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                 : "memory");
}

FA_DEVI void tc_fence_before_sync() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
FA_DEVI void tc_fence_after_sync() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
FA_DEVI void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
FA_DEVI void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Arrive (count 1) on an mbarrier once every tcgen05 async op issued so far by
// this thread has completed.  Implies tcgen05.fence::before_thread_sync.
FA_DEVI void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(bar) : "memory");
}

// ------------------------------------------------------------------ tcgen05: descriptors

// Instruction descriptor for kind::f16 with bf16 A/B and fp32 accumulation.
//   bits [4,6)  D format (1 = f32)        bits [7,10)  A format (1 = bf16)
//   bits [10,13) B format (1 = bf16)      bit 15 / 16  A / B major (0 = K-major, 1 = MN-major)
//   bits [17,23) N >> 3                   bits [24,29) M >> 4
__host__ __device__ constexpr uint32_t make_idesc_bf16_f32(int m, int n, bool a_mn_major, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) |
           ((b_mn_major ? 1u : 0u) << 16) | (static_cast<uint32_t>(n >> 3) << 17) |
           (static_cast<uint32_t>(m >> 4) << 24);
}

// Same fields for kind::f8f6f4 with e4m3 (format code 0) operands.
__host__ __device__ constexpr uint32_t make_idesc_e4m3_f32(int m, int n, bool a_mn_major, bool b_mn_major) {
    return (1u << 4) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
           (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}

// Shared-memory matrix descriptor, 128-byte swizzle.
//   bits [0,14)  start address >> 4       bits [16,30) leading byte offset >> 4
//   bits [32,46) stride byte offset >> 4  bits [46,48) version (1 on sm_100)
//   bits [61,64) layout (2 = 128-byte swizzle)
// K-major operand (rows of 64 bf16 = 128 B, 8-row groups 1024 B apart):
//   lbo is ignored for swizzled K-major layouts (set to 1), sbo = 1024.
// MN-major operand (rows = K index, 64 contiguous MN elements per row):
//   lbo = distance between 64-element MN chunks, sbo = distance between 8-row K groups.
FA_DEVI uint64_t make_smem_desc_sw128(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}

// ------------------------------------------------------------------ tcgen05: MMA

// D[tmem] (+)= A[smem] * B[smem]; issued by ONE thread.  accumulate = 0 overwrites D.
FA_DEVI void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                    uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// 8-bit operands (kind::f8f6f4): one instruction covers K = 32.  Measured on B200: 67 clk per
// 128x128x32, i.e. twice the bf16 rate; operands may be K-major or MN-major like the 16-bit ones.
FA_DEVI void mma_ss_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                       uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// A from TMEM: four e4m3 values per 32-bit column, lowest K index in the lowest byte.
FA_DEVI void mma_ts_f8(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                       uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Block-scaled 8-bit operands (kind::mxf8f6f4.block_scale): e4m3 data with one e8m0 scale (2^(byte - 127)) per
// 32 elements along K, for every row of A and every column of B; one instruction covers K = 32, i.e. one scale
// per row / column.  The scales sit in TMEM: a 128-row (or 128-column) operand takes 4 columns; lane l of every
// 32-lane quadrant holds, in column g and byte kb, the scale of row l % 32 + 32 g for K block kb, and the
// instruction descriptor names the byte (make_idesc_mx_e4m3's sf ids).  They get there from shared memory with
// tcgen05.cp 32x128b.warpx4 (32 rows of 16 bytes, replicated to the four quadrants), source bytes at
// (r % 32) * 16 + (r / 32) * 4 + kb.  Probed bit-exact on B200 with exactly representable data, both with A
// from shared memory and with A from TMEM and an MN-major B.
//   bits [4,6) B scale id   [7,10) A format (0 = e4m3)   [10,13) B format   15 / 16 A / B major
//   [17,23) N >> 3   23 scale format (1 = e8m0)   [24,29) M >> 4   [29,31) A scale id
__host__ __device__ constexpr uint32_t make_idesc_mx_e4m3(int m, int n, bool b_mn_major, uint32_t a_sf_id, uint32_t b_sf_id) {
    return (b_sf_id << 4) | ((b_mn_major ? 1u : 0u) << 16) | (static_cast<uint32_t>(n >> 3) << 17) | (1u << 23) |
           (static_cast<uint32_t>(m >> 4) << 24) | (a_sf_id << 29);
}
FA_DEVI void mma_ss_mx(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t sfa_tmem, uint32_t sfb_tmem,
                       uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
        : "memory");
}
FA_DEVI void mma_ts_mx(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t sfa_tmem, uint32_t sfb_tmem,
                       uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], [%1], %2, %3, [%5], [%6], p;\n"
        "}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
        : "memory");
}
// 32 rows x 16 bytes from shared memory into 4 TMEM columns of all four lane quadrants; issued by ONE thread, in
// order with that thread's MMAs (and covered by its next tcgen05.commit).  The source is described like a K-major
// MMA operand without swizzle: 8-row x 16-byte core matrices 128 bytes apart.
FA_DEVI void tmem_cp_scales_32x16B(uint32_t taddr, uint32_t saddr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>(16u >> 4) << 16;
    d |= static_cast<uint64_t>(128u >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(d) : "memory");
}
// Plain (untiled) bulk copy global -> shared with completion on an mbarrier; both addresses 16-byte aligned,
// size a multiple of 16.
FA_DEVI void bulk_load_1d(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem]; A holds bf16 pairs packed in 32-bit columns.
FA_DEVI void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                    uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// ------------------------------------------------------------------ tcgen05: ld / st (32x32b)
// Warp w of a warpgroup touches TMEM lanes 32*(w%4) .. 32*(w%4)+31; thread t of
// the warp gets lane 32*(w%4)+t, N consecutive 32-bit columns starting at the
// address's column.  The lane field of `taddr` must be 32*(w%4).

FA_DEVI void tmem_ld_x8(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7])
        : "r"(taddr)
        : "memory");
}

FA_DEVI void tmem_ld_x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]),
          "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

FA_DEVI void tmem_ld_x32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
          "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]),
          "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]),
          "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

FA_DEVI void tmem_st_x8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]),
          "r"(r[6]), "r"(r[7])
        : "memory");
}

FA_DEVI void tmem_st_x16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]),
          "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]),
          "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

FA_DEVI void tmem_st_x32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]),
          "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]),
          "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
          "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}

// ------------------------------------------------------------------ pairs of CTAs (cluster of two, tcgen05 cta_group::2)

FA_DEVI uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the variable that sits at `addr` (a shared::cta address) in CTA `rank` of the cluster
FA_DEVI uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// All threads of the cluster execute both.  The wait returns once every thread of the cluster that has not exited
// has arrived.
FA_DEVI void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
FA_DEVI void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// Arrive on an mbarrier of any CTA of the cluster (shared::cluster address).  The plain form, as for a local
// barrier: what is handed over with it here lives in TMEM and is ordered by the tcgen05 fences around the barrier
// (tcgen05.wait::st, tcgen05.fence::before_thread_sync on this side, fence::after_thread_sync on the waiter's).
// Measured on B200, round trip between the two CTAs of a pair: 359 cycles with this form and a plain try_wait, 943
// with .release.cluster on the arrive and .acquire.cluster on the wait.
FA_DEVI void mbar_arrive_cluster(uint32_t bar_cluster) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
FA_DEVI void st_shared_cluster_u32(uint32_t addr_cluster, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr_cluster), "r"(v) : "memory");
}
// 4-D tiled load into this CTA's shared memory whose bytes are counted on an mbarrier that may sit in the partner
// CTA (shared::cluster address).  Every CTA fetches its own box into its own shared memory.
FA_DEVI void tma_load_4d_2cta(uint32_t dst_smem, const CUtensorMap* map, uint32_t bar_cluster,
                              int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst_smem), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster),
          "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
// TMEM of both CTAs of a pair: warp w of BOTH CTAs executes each of these.
FA_DEVI void tmem_alloc_2cta(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_dst), "r"(ncols) : "memory");
}
FA_DEVI void tmem_relinquish_alloc_permit_2cta() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
FA_DEVI void tmem_dealloc_2cta(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
                 : "memory");
}
// Arrive (count 1) on the mbarrier at this offset in BOTH CTAs of the pair once every tcgen05 async op issued so far
// by this thread has completed: one commit per CTA, the partner's barrier through its mapped address.
FA_DEVI void tc_commit_2cta(uint32_t bar, uint32_t bar_in_partner) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_in_partner) : "memory");
}
// 256 x N x 16 MMAs over a CTA pair, issued by ONE thread of the even CTA: rows 0..127 of A and D belong to the
// even CTA, rows 128..255 to the odd one; each CTA supplies N/2 columns of B from its own shared memory (same
// offsets in both CTAs).
FA_DEVI void mma2_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
FA_DEVI void mma2_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// One asm statement: probe up to three mbarriers, issue three SS MMAs (all accumulating),
// then read the probes' predicates; bit i of the result = probe i found its phase complete.
FA_DEVI uint32_t probe3_mma2_ss3(uint32_t bar0, uint32_t par0, uint32_t bar1, uint32_t par1, uint32_t bar2, uint32_t par2,
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
        "tcgen05.mma.cta_group::2.kind::f16 [%7], %8, %9, %14, q;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%7], %10, %11, %14, q;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%7], %12, %13, %14, q;\n"
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
FA_DEVI uint32_t probe_mma2_ts2(uint32_t bar, uint32_t par, uint32_t d_tmem, uint32_t a0_tmem, uint64_t b0, uint32_t a1_tmem,
                                uint64_t b1, uint32_t idesc) {
    uint32_t r;
    asm volatile(
        "{\n"
        ".reg .pred p0, q;\n"
        "setp.ne.b32 q, 1, 0;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p0, [%1], %2;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%3], [%4], %5, %8, q;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%3], [%6], %7, %8, q;\n"
        "selp.u32 %0, 1, 0, p0;\n"
        "}\n"
        : "=r"(r)
        : "r"(bar), "r"(par), "r"(d_tmem), "r"(a0_tmem), "l"(b0), "r"(a1_tmem), "l"(b1), "r"(idesc)
        : "memory");
    return r;
}

}  // namespace ptx
}  // namespace fa
