// Types shared by the attention forward kernels and the host-side launcher.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace fa {

constexpr int kTileM = 128;       // query rows per tile (one TMEM lane per row)
constexpr int kTileN = 128;       // keys per K/V tile
constexpr int kChunkCols = 64;    // bf16 columns per 128-byte swizzled smem row
constexpr int kChunkBytes = kTileN * kChunkCols * 2;   // one 128-row x 64-col chunk = 16 KB

// "who" codes recorded when a bounded wait gives up: (role << 8) | barrier id.
enum WaitSite : uint32_t {
    kSiteSimpleQ = 0x0101, kSiteSimpleK = 0x0102, kSiteSimpleV = 0x0103, kSiteSimpleMma = 0x0104,
    kSiteLoadKvEmpty = 0x0201, kSiteLoadQEmpty = 0x0202,
    kSiteMmaQFull = 0x0301, kSiteMmaKvFull = 0x0302, kSiteMmaPFull = 0x0303,
    kSiteMmaOReady = 0x0304, kSiteMmaSFree = 0x0305, kSiteMmaTurn = 0x0306,
    kSiteSoftmaxSFull = 0x0401, kSiteSoftmaxPFree = 0x0402, kSiteSoftmaxCorrFree = 0x0403,
    kSiteCorrScale = 0x0501, kSiteCorrPvDone = 0x0502, kSiteCorrFinal = 0x0503,
    kSiteEpiOFull = 0x0601, kSiteEpiStaged = 0x0602, kSiteEpiState = 0x0603,
    kSiteSmemAlign = 0x0701,
    kSiteItem = 0x0801,
};

struct FwdParams {
    __nv_bfloat16* O;         // element (b, hq, i, c) at O + b*o_stride_b + hq*o_stride_h + i*o_stride_s + c
    long long o_stride_b, o_stride_h, o_stride_s;   // in elements
    float* lse;               // [B, Hq, Sq] or nullptr
    int B, Hq, Hkv, Sq, Sk;
    // Variable-length batches: sequence b owns rows [cu_q[b], cu_q[b+1]) of the packed Q/O and
    // [cu_k[b], cu_k[b+1]) of the packed K/V (device arrays of B+1 ints); nullptr = fixed Sq/Sk.
    // Then Sq is the longest query length (grid sizing only) and lse is [Hq, total_q].
    const int* cu_q;
    const int* cu_k;
    int total_q;
    int causal;
    float scale_log2;         // scale * log2(e): scores are handled in log2 units
    int n_q_tiles;            // ceil(Sq / 128)
    int heads_per_group;      // (batch, head) instances scheduled together (their K/V share L2)
    int kv_splits;            // C >= 1: CTAs per item, each with its own range of K/V tiles
    int tiles_per_split;      // K/V tiles per split (all of them when kv_splits == 1)
    int pack_heads;           // query heads of one K/V head sharing a query tile (stream kernels with kPack; else unused)
    int head_pair;            // persistent kernel: 1 = an item is one query tile of two adjacent heads of a group
    float* o_part;            // [C, B*Hq, Sq, dv] fp32 partial outputs (split-KV only)
    float* lse_part;          // [C, B*Hq, Sq] fp32 partial log-sum-exps (split-KV only)
    int debug_drop_v_load;    // test hook: the load warp skips the first V tile (exercises the wait limit)
    unsigned int* sched_counter;   // persistent kernel: ticket counter of the work-item list (zero between launches)
    uint32_t* status;         // [0] = fa_status, [1] = wait site; mapped host memory
    unsigned long long wait_limit_ns;
#ifdef FA_TRACE
    long long* trace;         // [role][iteration][event] SM clock stamps of CTA (0,0,0); debug builds only
#endif
};

#ifdef FA_TRACE
constexpr int kTraceIters = 64, kTraceEvents = 16, kTraceRoles = 6;   // roles: softmax0, softmax1, mma, corr
#endif
// -DFA_TRACE alone records one (SM, start, end, rounds) entry per CTA; -DFA_TRACE_STAMPS adds the
// per-iteration clock stamps of CTA 0 (they cost a few hundred cycles each and slow the loop).
#if defined(FA_TRACE) && defined(FA_TRACE_STAMPS)
#define FA_TRACE_STAMP(role, iter, ev)                                                          \
    do {                                                                                        \
        if (p.trace && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && (iter) < kTraceIters) \
            p.trace[((role) * kTraceIters + (iter)) * kTraceEvents + (ev)] = clock64();         \
    } while (0)
#else
#define FA_TRACE_STAMP(role, iter, ev) do { } while (0)
#endif

// -DFA_TRACE -DFA_TRACE_PHASES: every softmax warp of the pair kernel adds up the cycles it spends in each part of
// its loop (clock reads at the points where the warp synchronises anyway) and leaves the sums in the trace buffer.
#if defined(FA_TRACE) && defined(FA_TRACE_PHASES)
#define FA_PHASE_DECL() uint32_t ph_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}, ph_last; asm volatile("mov.u32 %0, %%clock;" : "=r"(ph_last))
#define FA_PHASE(k) do { uint32_t c_; asm volatile("mov.u32 %0, %%clock;" : "=r"(c_)); ph_acc[k] += c_ - ph_last; ph_last = c_; } while (0)
#define FA_PHASE_STORE(nphases, count)                                                                       \
    do {                                                                                                     \
        if (lane == 0 && p.trace) {                                                                          \
            uint32_t* o_ = reinterpret_cast<uint32_t*>(p.trace) + (static_cast<size_t>(blockIdx.x) * 16 + warp) * 8; \
            for (int k_ = 0; k_ < (nphases); ++k_) o_[k_] = ph_acc[k_];                                      \
            o_[7] = (count);                                                                                 \
        }                                                                                                    \
    } while (0)
#else
#define FA_PHASE_DECL() do { } while (0)
#define FA_PHASE(k) do { } while (0)
#define FA_PHASE_STORE(nphases, count) do { } while (0)
#endif

// Number of K/V tiles a query tile starting at row i0 (covering `rows` rows) has to visit.
// Key j is visible to query i iff j <= i + (Sk - Sq) in causal mode.
__host__ __device__ inline int kv_tiles_for_q_tile(int i0, int rows, int Sq, int Sk, int causal) {
    int last_key = Sk - 1;
    if (causal) {
        int last_row = i0 + rows - 1;
        if (last_row > Sq - 1) last_row = Sq - 1;
        const int lim = last_row + (Sk - Sq);
        if (lim < last_key) last_key = lim;
    }
    return last_key < 0 ? 0 : last_key / kTileN + 1;
}

}  // namespace fa
