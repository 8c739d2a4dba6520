// Host side of the C ABI declared in include/fa.h: argument checks, TMA tensor
// maps, kernel selection and launch.  No torch types, no CPU fallback.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "../../include/fa.h"
#include "fa_common.cuh"
#include "fa_fwd_pipelined.cuh"
#include "fa_fwd_pair.cuh"
#include "fa_fwd_duo.cuh"
#include "fa_fwd_quad.cuh"
#include "fa_fwd_stream_persistent.cuh"
#include "fa_fwd_pair_persistent.cuh"
#include "fa_fwd_persistent.cuh"
#include "fa_fwd_stream.cuh"
#include "fa_fwd_fp8.cuh"
#include "fa_fwd_fp8_stream.cuh"
#include "fa_fwd_simple.cuh"

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct MapEntry {
    const void* ptr;
    int d, S, H, B, box_rows, box_heads, elem_bytes, swizzle_bytes;
    long long sb, sh, ss;      // batch / head / row strides in elements
    uint64_t stamp;
    CUtensorMap map;
};

constexpr int kMapCacheSize = 16;

}  // namespace

struct fa_handle {
    int device = 0;
    int num_sms = 1;
    uint32_t flags = 0;
    uint32_t* status_host = nullptr;   // pinned + mapped: [0] status, [1] wait site
    uint32_t* status_dev = nullptr;
    uint32_t kv_splits_cfg = 0;              // 0 auto, 1 never, n force
    void* scratch = nullptr;                 // split-KV partials
    unsigned int* sched_counter = nullptr;   // work-item ticket counter of the persistent kernel
    size_t scratch_bytes = 0;
    int last_splits = 1;
    unsigned long long wait_limit_ns = 2000ull * 1000000ull;
    EncodeTiledFn encode = nullptr;
    std::vector<MapEntry> maps;
    uint64_t stamp = 0;
    uint64_t launches = 0;
    const char* last_kernel = "";
    void* stage[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};   // Q K V O lse
    size_t stage_cap[5] = {0, 0, 0, 0, 0};
    // fa_forward_host on large problems: copy streams and events of the chunked pipeline (created on first use)
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_out_done = nullptr;
    std::vector<cudaEvent_t> ev_in, ev_done;
    std::vector<const void*> attr_done;     // kernels whose shared-memory limit has been raised
#ifdef FA_TRACE
    long long* trace = nullptr;
#endif
};

namespace {

class DeviceGuard {
  public:
    explicit DeviceGuard(int want) {
        if (cudaGetDevice(&prev_) != cudaSuccess) prev_ = -1;
        if (prev_ != want) { ok_ = (cudaSetDevice(want) == cudaSuccess); changed_ = ok_; }
    }
    ~DeviceGuard() { if (changed_ && prev_ >= 0) cudaSetDevice(prev_); }
    bool ok() const { return ok_; }
  private:
    int prev_ = -1;
    bool ok_ = true;
    bool changed_ = false;
};

// Tensor of bf16 (elem_bytes 2) or e4m3 (elem_bytes 1) with element (b, h, s, c) at
// ptr + b*sb + h*sh + s*ss + c, seen as a 4-D TMA tensor (d, S, H, B); box = 128 bytes of columns
// x box_rows rows, 128-byte swizzle, rows past S read as zero.
fa_status get_map(fa_handle* h, const void* ptr, int d, int S, int H, int B, long long sb, long long sh,
                  long long ss, int box_rows, const CUtensorMap** out, int elem_bytes = 2, int box_heads = 1,
                  int swizzle_bytes = 128) {
    for (auto& e : h->maps) {
        if (e.ptr == ptr && e.d == d && e.S == S && e.H == H && e.B == B && e.box_rows == box_rows &&
            e.sb == sb && e.sh == sh && e.ss == ss && e.elem_bytes == elem_bytes && e.box_heads == box_heads && e.swizzle_bytes == swizzle_bytes) {
            e.stamp = ++h->stamp;
            *out = &e.map;
            return FA_OK;
        }
    }
    MapEntry ne;
    memset(&ne, 0, sizeof ne);
    ne.ptr = ptr; ne.d = d; ne.S = S; ne.H = H; ne.B = B; ne.box_rows = box_rows;
    ne.sb = sb; ne.sh = sh; ne.ss = ss; ne.elem_bytes = elem_bytes; ne.box_heads = box_heads; ne.swizzle_bytes = swizzle_bytes;
    const cuuint64_t eb = static_cast<cuuint64_t>(elem_bytes);
    const cuuint64_t dims[4] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(S),
                                static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(B)};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(ss) * eb, static_cast<cuuint64_t>(sh) * eb,
                                   static_cast<cuuint64_t>(sb) * eb};
    const cuuint32_t box[4] = {static_cast<cuuint32_t>(swizzle_bytes / elem_bytes), static_cast<cuuint32_t>(box_rows),
                              static_cast<cuuint32_t>(box_heads), 1u};
    const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    const CUresult r = h->encode(&ne.map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8,
                                 4, const_cast<void*>(ptr),
                                 dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                 swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return FA_ERR_INVALID_ARG;     // strides or extents the TMA unit cannot express
    ne.stamp = ++h->stamp;
    if (static_cast<int>(h->maps.size()) < kMapCacheSize) {
        h->maps.push_back(ne);
        *out = &h->maps.back().map;
    } else {
        size_t victim = 0;
        for (size_t i = 1; i < h->maps.size(); ++i)
            if (h->maps[i].stamp < h->maps[victim].stamp) victim = i;
        h->maps[victim] = ne;
        *out = &h->maps[victim].map;
    }
    return FA_OK;
}

// Raises a kernel's dynamic shared-memory limit once per handle (the attribute is per device and
// function; the handle remembers which kernels it has prepared, by their address).
template <typename Kernel>
fa_status ensure_smem_attr(fa_handle* h, Kernel kernel, int bytes) {
    const void* key = reinterpret_cast<const void*>(kernel);
    for (const void* k : h->attr_done)
        if (k == key) return FA_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) {
        cudaGetLastError();
        return FA_ERR_CUDA;
    }
    h->attr_done.push_back(key);
    return FA_OK;
}

template <int DQK, int DV>
fa_status launch_simple(fa_handle* h, const CUtensorMap& mq, const CUtensorMap& mk,
                        const CUtensorMap& mv, const fa::FwdParams& p, cudaStream_t st) {
    using Cfg = fa::SimpleCfg<DQK, DV>;
    // ask for more than half of the SM's shared memory so that one CTA owns the SM's TMEM
    const int smem = Cfg::kSmemBytes > 120 * 1024 ? Cfg::kSmemBytes : 120 * 1024;
    auto kernel = fa::fa_fwd_simple_kernel<DQK, DV>;
    fa_status s = ensure_smem_attr(h, kernel, smem);
    if (s != FA_OK) return s;
    dim3 grid(p.n_q_tiles, p.Hq, p.B);
    kernel<<<grid, 128, smem, st>>>(mq, mk, mv, p);
    if (cudaGetLastError() != cudaSuccess) return FA_ERR_CUDA;
    h->launches += 1;
    return FA_OK;
}

// Launch of a kernel with two query tiles per CTA (and of the combine kernel behind it with split-KV).
template <int DV, typename Kernel>
fa_status launch_two_tile(fa_handle* h, Kernel kernel, int smem, int threads, bool head_pair, const CUtensorMap& mq,
                          const CUtensorMap& mk, const CUtensorMap& mv, const CUtensorMap& mo, const fa::FwdParams& p,
                          cudaStream_t st) {
    fa_status s = ensure_smem_attr(h, kernel, smem);
    if (s != FA_OK) return s;
    // items: pairs of adjacent query tiles of a head, or one query tile of a pair of adjacent heads
    const long long n_ctas = (head_pair ? static_cast<long long>(p.n_q_tiles) * (p.Hq / 2)
                                        : static_cast<long long>((p.n_q_tiles + 1) / 2) * p.Hq) * p.B * p.kv_splits;
    if (n_ctas > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;
    // Programmatic stream serialisation: the kernel may be scheduled while its predecessor in the
    // stream drains (both kernels wait for that predecessor's completion before they touch global
    // memory); without it every launch pays the full completion-to-launch latency of the stream.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(n_ctas), 1, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = (h->flags & FA_FLAG_NO_DEPENDENT_LAUNCH) ? 0 : 1;
    if (cudaLaunchKernelEx(&cfg, kernel, mq, mk, mv, mo, p) != cudaSuccess) return FA_ERR_CUDA;
    h->launches += 1;
    if (p.kv_splits > 1) {
        const long long n_rows = static_cast<long long>(p.B) * p.Hq * p.Sq;
        const long long blocks = (n_rows + 3) / 4;
        if (blocks > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;
        cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
        cfg.blockDim = dim3(128, 1, 1);
        cfg.dynamicSmemBytes = 0;
        if (cudaLaunchKernelEx(&cfg, fa::fa_combine_kernel<DV>, static_cast<const float*>(p.o_part),
                               static_cast<const float*>(p.lse_part), p.O, p.lse, n_rows, p.kv_splits, p.Hq, p.Sq,
                               p.o_stride_b, p.o_stride_h, p.o_stride_s) != cudaSuccess) return FA_ERR_CUDA;
        h->launches += 1;
    }
    return FA_OK;
}

// Two query tiles per CTA, one item per CTA: at head size 128 the kernel of fa_fwd_pair.cuh, otherwise
// (and with FA_FLAG_LEGACY_PAIR_KERNEL) the one of fa_fwd_pipelined.cuh.
template <int DQK, int DV, bool kVarlen, bool kHeadPair = false>
fa_status launch_pipelined(fa_handle* h, const CUtensorMap& mq, const CUtensorMap& mk,
                           const CUtensorMap& mv, const CUtensorMap& mo, const fa::FwdParams& p, cudaStream_t st) {
    if constexpr (DQK == 128 && DV == 128) {
        if (!(h->flags & FA_FLAG_LEGACY_PAIR_KERNEL)) {
            constexpr int smem = fa::pair_smem_bytes<DQK, DV>();
            static_assert(smem <= 227 * 1024, "shared memory budget exceeded");
            h->last_kernel = "fa_fwd_pair";
            return launch_two_tile<DV>(h, fa::fa_fwd_pair_kernel<DQK, DV, kVarlen, kHeadPair>, smem,
                                       fa::PairCfg<DQK, DV>::kThreads, kHeadPair, mq, mk, mv, mo, p, st);
        }
    }
    constexpr int smem = fa::pipe_smem_bytes<DQK, DV>();
    static_assert(smem <= 227 * 1024, "shared memory budget exceeded");
    return launch_two_tile<DV>(h, fa::fa_fwd_pipelined_kernel<DQK, DV, kVarlen, kHeadPair>, smem,
                               fa::PipeCfg<DQK, DV>::kThreads, kHeadPair, mq, mk, mv, mo, p, st);
}

// One query tile per CTA on pairs of CTAs (clusters of two, two-CTA MMAs): fa_fwd_duo.cuh.
template <int DQK, int DV, bool kHeadPair>
fa_status launch_duo(fa_handle* h, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                     const CUtensorMap& mo, const fa::FwdParams& p, cudaStream_t st) {
    constexpr int smem = fa::duo_smem_bytes<DQK, DV>();
    static_assert(smem <= 227 * 1024, "shared memory budget exceeded");
    auto kernel = fa::fa_fwd_duo_kernel<DQK, DV, kHeadPair>;
    fa_status s = ensure_smem_attr(h, kernel, smem);
    if (s != FA_OK) return s;
    // one cluster per item: two adjacent query tiles of a head, or one query tile of two adjacent heads
    const long long n_ctas = 2 * (kHeadPair ? static_cast<long long>(p.n_q_tiles) * (p.Hq / 2)
                                            : static_cast<long long>((p.n_q_tiles + 1) / 2) * p.Hq) * p.B;
    if (n_ctas > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(n_ctas), 1, 1);       // the kernel carries __cluster_dims__(2, 1, 1)
    cfg.blockDim = dim3(fa::DuoCfg<DQK, DV>::kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = (h->flags & FA_FLAG_NO_DEPENDENT_LAUNCH) ? 0 : 1;
    if (cudaLaunchKernelEx(&cfg, kernel, mq, mk, mv, mo, p) != cudaSuccess) return FA_ERR_CUDA;
    h->launches += 1;
    return FA_OK;
}

// Four query tiles per pair of CTAs (clusters of two, two-CTA MMAs, two tiles per CTA): fa_fwd_quad.cuh.
template <int DQK, int DV, int kMode>
fa_status launch_quad(fa_handle* h, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                      const CUtensorMap& mo, const fa::FwdParams& p, cudaStream_t st) {
    constexpr int smem = fa::quad_smem_bytes<DQK, DV>();
    static_assert(smem <= 227 * 1024, "shared memory budget exceeded");
    auto kernel = fa::fa_fwd_quad_kernel<DQK, DV, kMode>;
    fa_status s = ensure_smem_attr(h, kernel, smem);
    if (s != FA_OK) return s;
    constexpr int heads = kMode == 0 ? 1 : (kMode == 1 ? 2 : 4);      // heads of an item; 4 / heads adjacent tiles of each
    const long long n_ctas = 2ll * ((p.n_q_tiles + 4 / heads - 1) / (4 / heads)) * (p.Hq / heads) * p.B;
    if (n_ctas > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(n_ctas), 1, 1);       // the kernel carries __cluster_dims__(2, 1, 1)
    cfg.blockDim = dim3(fa::QuadCfg<DQK, DV>::kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = (h->flags & FA_FLAG_NO_DEPENDENT_LAUNCH) ? 0 : 1;
    if (cudaLaunchKernelEx(&cfg, kernel, mq, mk, mv, mo, p) != cudaSuccess) return FA_ERR_CUDA;
    h->launches += 1;
    return FA_OK;
}

// Number of K/V splits for a problem: 1 unless the query tiles alone leave most SMs idle and the
// K/V range is long enough to cut; never more than the scratch buffer can hold partials for.
int choose_kv_splits(int num_sms, uint32_t kv_splits_cfg, size_t scratch_bytes, int B, int Hq, int Sq, int Sk, int dv,
                     int causal, int n_q_tiles, bool one_tile_items = false, int heads_per_item = 1) {
    const long long items = static_cast<long long>(one_tile_items ? n_q_tiles : (n_q_tiles + 1) / 2) * B * (Hq / heads_per_item);
    int max_tiles = fa::kv_tiles_for_q_tile((n_q_tiles - 1) * fa::kTileM, fa::kTileM, Sq, Sk, causal);
    if (!causal) max_tiles = (Sk + fa::kTileN - 1) / fa::kTileN;
    int splits = 1;
    if (kv_splits_cfg == 1) return 1;
    if (kv_splits_cfg > 1) {
        splits = static_cast<int>(kv_splits_cfg);
    } else if (items * 2 <= num_sms && max_tiles >= 8) {
        // One wave at most.  Inside that, a split costs about 0.3 us (its partial, its share of the
        // merge) and saves 1 us per K/V tile it takes off the longest CTA: a * tiles / C + b * C
        // is least at C = sqrt(a * tiles / b); equal shares matter as much, so C is a power of two
        // (measured optimum 4 / 8 / 8 / 16 for 8 / 16 / 32 / 64 tiles) and splits that would get
        // no tile are not launched.
        const int wave = static_cast<int>(num_sms / items);
        const double ideal = sqrt(3.3 * max_tiles);
        splits = 1;
        while (splits * 2 <= wave && splits * 2 <= 128 && splits * 1.41 < ideal) splits *= 2;
        const int per_split = (max_tiles + splits - 1) / splits;
        splits = (max_tiles + per_split - 1) / per_split;
    }
    if (splits > max_tiles) splits = max_tiles;
    if (splits < 1) splits = 1;
    const long long rows = static_cast<long long>(B) * Hq * Sq;
    while (splits > 1 && static_cast<unsigned long long>(splits) * rows * (dv + 1) * 4ull > scratch_bytes) --splits;
    return splits;
}

bool misaligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }

fa_status check_args(const void* Q, const void* K, const void* V, const void* O, const float* lse,
                     int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv, float scale,
                     bool device_ptrs) {
    if (!Q || !K || !V || !O) return FA_ERR_INVALID_ARG;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || dqk <= 0 || dv <= 0)
        return FA_ERR_INVALID_ARG;
    if (Hq % Hkv != 0) return FA_ERR_INVALID_ARG;
    if (!isfinite(scale) || scale < 0.f) return FA_ERR_INVALID_ARG;
    if (device_ptrs) {
        if (misaligned(Q, 16) || misaligned(K, 16) || misaligned(V, 16) || misaligned(O, 16))
            return FA_ERR_INVALID_ARG;
        if (lse && misaligned(lse, 4)) return FA_ERR_INVALID_ARG;
    }
    const bool dims_ok = (dqk == 64 && dv == 64) || (dqk == 128 && dv == 128) || (dqk == 192 && dv == 128);
    if (!dims_ok) return FA_ERR_UNSUPPORTED;
    const long long n_q_tiles = (static_cast<long long>(Sq) + fa::kTileM - 1) / fa::kTileM;
    if (Hq > 65535 || B > 65535 || n_q_tiles > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;
    if (static_cast<long long>(B) * Hq > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;
    return FA_OK;
}

// Number of (batch, query head) instances scheduled together.  The K and V of a group (read again
// by every query tile of its heads) should fit in about a third of the 126 MB L2, a group holds
// whole GQA groups, and the groups are made equal in size: a small last group would start its
// longest items late and leave most SMs idle under them.
int heads_per_group(long long kv_bytes_per_head, int B, int Hq, int Hkv) {
    const long long budget = 48ll << 20;      // 32 to 96 MB measure the same within 2 %
    long long kv_heads = budget / kv_bytes_per_head;
    if (kv_heads < 1) kv_heads = 1;
    const long long gqa = Hq / Hkv;
    const long long n_kv = static_cast<long long>(B) * Hkv;       // K/V heads in the batch
    if (kv_heads > n_kv) kv_heads = n_kv;
    const long long n_groups = (n_kv + kv_heads - 1) / kv_heads;
    kv_heads = (n_kv + n_groups - 1) / n_groups;
    return static_cast<int>(kv_heads * gqa);
}

// Persistent kernel: one CTA per SM (fewer when there are fewer items), every CTA walks its share
// of the items.  No split-KV.
template <int DQK, int DV, bool kVarlen = false>
fa_status launch_persistent(fa_handle* h, const CUtensorMap& mq, const CUtensorMap& mk,
                            const CUtensorMap& mv, const CUtensorMap& mo, const fa::FwdParams& p, cudaStream_t st) {
    const long long n_items = p.head_pair ? static_cast<long long>(p.n_q_tiles) * (p.Hq / 2) * p.B
                                          : static_cast<long long>((p.n_q_tiles + 1) / 2) * p.Hq * p.B;
    if (n_items > 0x3fffffffLL) return FA_ERR_UNSUPPORTED;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(n_items < h->num_sms ? n_items : h->num_sms), 1, 1);
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = (h->flags & FA_FLAG_NO_DEPENDENT_LAUNCH) ? 0 : 1;
    if constexpr (DQK == 128 && DV == 128) {
        // head size 128: the persistent form of the kernel of fa_fwd_pair.cuh (FA_FLAG_LEGACY_PAIR_KERNEL: the earlier one)
        if (!(h->flags & FA_FLAG_LEGACY_PAIR_KERNEL)) {
            constexpr int smem = fa::pair_persist_smem_bytes();
            static_assert(smem <= 227 * 1024, "shared memory budget exceeded");
            auto kernel = fa::fa_fwd_pair_persistent_kernel<kVarlen>;
            fa_status s = ensure_smem_attr(h, kernel, smem);
            if (s != FA_OK) return s;
            cfg.blockDim = dim3(fa::PairPersistCfg::kThreads, 1, 1);
            cfg.dynamicSmemBytes = smem;
            if (cudaLaunchKernelEx(&cfg, kernel, mq, mk, mv, mo, p) != cudaSuccess) return FA_ERR_CUDA;
            h->launches += 1;
            return FA_OK;
        }
    }
    constexpr int smem = fa::persist_smem_bytes<DQK, DV>();
    static_assert(smem <= 227 * 1024, "shared memory budget exceeded");
    auto kernel = fa::fa_fwd_persistent_kernel<DQK, DV, kVarlen>;
    fa_status s = ensure_smem_attr(h, kernel, smem);
    if (s != FA_OK) return s;
    cfg.blockDim = dim3(fa::PipeCfg<DQK, DV>::kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    if (cudaLaunchKernelEx(&cfg, kernel, mq, mk, mv, mo, p) != cudaSuccess) return FA_ERR_CUDA;
    h->launches += 1;
    return FA_OK;
}

// One query tile per CTA, K/V tiles streamed through two softmax warpgroups.
template <int DQK, int DV, bool kVarlen = false, bool kPack = false>
fa_status launch_stream(fa_handle* h, const CUtensorMap& mq, const CUtensorMap& mk,
                        const CUtensorMap& mv, const CUtensorMap& mo, const fa::FwdParams& p, cudaStream_t st) {
    constexpr int smem = fa::stream_smem_bytes<DQK, DV>();
    static_assert(smem <= 227 * 1024, "shared memory budget exceeded");
    auto kernel = fa::fa_fwd_stream_kernel<DQK, DV, kVarlen, kPack>;
    fa_status s = ensure_smem_attr(h, kernel, smem);
    if (s != FA_OK) return s;
    // items: query tiles x heads, or packs of heads with their single query tile
    const long long n_ctas = (kPack ? static_cast<long long>(p.Hq / p.pack_heads) : static_cast<long long>(p.n_q_tiles) * p.Hq) * p.B * p.kv_splits;
    if (n_ctas > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(n_ctas), 1, 1);
    cfg.blockDim = dim3(512, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = (h->flags & FA_FLAG_NO_DEPENDENT_LAUNCH) ? 0 : 1;
    if (cudaLaunchKernelEx(&cfg, kernel, mq, mk, mv, mo, p) != cudaSuccess) return FA_ERR_CUDA;
    h->launches += 1;
    if (p.kv_splits > 1) {
        // packed batches are one batch slice of total_q rows per head ([Hq, total_q] partials and lse)
        const int rows_per_head = kVarlen ? p.total_q : p.Sq;
        const long long n_rows = static_cast<long long>(kVarlen ? 1 : p.B) * p.Hq * rows_per_head;
        const long long blocks = (n_rows + 3) / 4;
        if (blocks > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;
        cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
        cfg.blockDim = dim3(128, 1, 1);
        cfg.dynamicSmemBytes = 0;
        if (cudaLaunchKernelEx(&cfg, fa::fa_combine_kernel<DV>, static_cast<const float*>(p.o_part),
                               static_cast<const float*>(p.lse_part), p.O, p.lse, n_rows, p.kv_splits, p.Hq, rows_per_head,
                               p.o_stride_b, p.o_stride_h, p.o_stride_s) != cudaSuccess) return FA_ERR_CUDA;
        h->launches += 1;
    }
    return FA_OK;
}

// Persistent form of the stream kernel: one CTA per SM (fewer when there are fewer items), every CTA walks its share of
// the (query tile, head) items in a fixed order.  Fixed lengths, no split-KV, no shared query tiles.
template <int DQK, int DV>
fa_status launch_stream_persistent(fa_handle* h, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                                   const CUtensorMap& mo, const fa::FwdParams& p, cudaStream_t st) {
    constexpr int smem = fa::stream_persist_smem_bytes<DQK, DV>();
    static_assert(smem <= 227 * 1024, "shared memory budget exceeded");
    auto kernel = fa::fa_fwd_stream_persistent_kernel<DQK, DV>;
    fa_status s = ensure_smem_attr(h, kernel, smem);
    if (s != FA_OK) return s;
    const long long n_items = static_cast<long long>(p.n_q_tiles) * p.Hq * p.B;
    if (n_items > 0x3fffffffLL) return FA_ERR_UNSUPPORTED;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(n_items < h->num_sms ? n_items : h->num_sms), 1, 1);
    cfg.blockDim = dim3(512, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = (h->flags & FA_FLAG_NO_DEPENDENT_LAUNCH) ? 0 : 1;
    if (cudaLaunchKernelEx(&cfg, kernel, mq, mk, mv, mo, p) != cudaSuccess) return FA_ERR_CUDA;
    h->launches += 1;
    return FA_OK;
}

// Estimated run times (microseconds) of a launch under the two tilings, from the measured cost of
// a CTA: pair kernel a_p * rounds + f_p with rounds = K/V tiles of the pair's second query tile
// (split-KV: rounds / C, plus the combine kernel); stream kernel a_s * (K/V tiles of the query tile)
// + f_s.  Longest-first scheduling over the SMs is approximated by max(longest item, total / SMs),
// and by whole waves when all items are equal.  Good to some 20 % on the shapes it was checked
// on, which is enough to tell a grid of under one wave (the stream kernel's case) from the rest.
struct TilingEstimate { double pair_us, stream_us; };
TilingEstimate estimate_tilings(int num_sms, int B, int Hq, int Sq, int Sk, int dqk, int causal, int n_q_tiles, int splits,
                                int stream_splits, bool head_pair) {
    // (at d_qk = 192 the pair kernel only has room for two K stages and one V stage and a longer MMA
    // chain per round; the stream kernel is ahead there at every size measured)
    const double a_p = dqk == 64 ? 1.36 : (dqk == 128 ? 2.0 : 2.9), f_p = dqk == 64 ? 6.0 : 6.7;
    const double a_s = dqk == 64 ? 0.75 : (dqk == 128 ? 1.0 : 1.05), f_s = 5.0;
    const double heads = static_cast<double>(B) * Hq;
    double pair_total = 0, pair_max = 0, stream_total = 0, stream_max = 0;
    for (int t = 0; t < n_q_tiles; ++t) {
        const int r = fa::kv_tiles_for_q_tile(t * fa::kTileM, fa::kTileM, Sq, Sk, causal);
        const double cs = a_s * ((r + stream_splits - 1) / stream_splits) + f_s;
        stream_total += cs * stream_splits;
        if (cs > stream_max) stream_max = cs;
        if (head_pair) {                                  // every query tile is an item of two heads
            const double cp = a_p * r + f_p;
            pair_total += 0.5 * cp;
            if (cp > pair_max) pair_max = cp;
        } else if ((t & 1) == 1 || t == n_q_tiles - 1) {  // second tile of a pair, or an unpaired last tile
            const double rounds = (r + splits - 1) / splits;
            const double cp = a_p * rounds + f_p;
            pair_total += cp * splits;
            if (cp > pair_max) pair_max = cp;
        }
    }
    auto makespan = [&](double total_per_head, double longest, double n_items_per_head) {
        const double n_items = n_items_per_head * heads;
        if (!causal && Sq >= fa::kTileM) {                // equal items: whole waves
            const double waves = static_cast<double>((static_cast<long long>(n_items) + num_sms - 1) / num_sms);
            return waves * longest;
        }
        const double balanced = total_per_head * heads / num_sms;
        return balanced > longest ? balanced : longest;
    };
    TilingEstimate e;
    e.pair_us = makespan(pair_total, pair_max, head_pair ? 0.5 * n_q_tiles : static_cast<double>((n_q_tiles + 1) / 2) * splits) +
                (splits > 1 ? 6.0 : 0.0);
    e.stream_us = makespan(stream_total, stream_max, static_cast<double>(n_q_tiles) * stream_splits) + (stream_splits > 1 ? 6.0 : 0.0);
    return e;
}

// Which kernel a launch uses and how its K/V range is split: a pure function of the problem, the
// handle's configuration and the SM count (fa_plan exposes it).
enum PlanKernel { kPlanSerial = 0, kPlanPair = 1, kPlanPersistent = 2, kPlanStream = 3, kPlanDuo = 4, kPlanQuad = 5, kPlanStreamPersistent = 6 };
struct LaunchPlan {
    int kernel;
    int kv_splits;
    int tiles_per_split;
    int pack_heads;                // > 1: stream kernel with that many query heads of a K/V head per query tile
    int quad_mode;                 // quad kernel: which four tiles a cluster takes (fa_fwd_quad.cuh)
    bool head_pair;                // pair kernel: the CTA's two tiles are one query tile of two adjacent heads of a group
    double pair_us, stream_us;     // the two estimates (0 when no estimate was needed)
};
// (packed batches: Sq is the longest query length, Sk the mean K/V length)
LaunchPlan plan_launch(int num_sms, uint32_t flags, uint32_t kv_splits_cfg, size_t scratch_bytes, bool varlen,
                       int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv, int causal) {
    LaunchPlan pl;
    pl.kernel = kPlanPair;
    pl.kv_splits = 1;
    pl.tiles_per_split = 0x3fffffff;
    pl.pack_heads = 1;
    pl.head_pair = false;
    pl.quad_mode = 0;
    pl.pair_us = pl.stream_us = 0.0;
    const int n_q_tiles = (Sq + fa::kTileM - 1) / fa::kTileM;
    int max_tiles = (Sk + fa::kTileN - 1) / fa::kTileN;           // K/V tiles of the longest query tile
    if (causal) {
        const int t = fa::kv_tiles_for_q_tile((n_q_tiles - 1) * fa::kTileM, fa::kTileM, Sq, Sk, 1);
        if (t < max_tiles) max_tiles = t;
    }
    auto with_splits = [&](int splits) {
        pl.kv_splits = splits;
        pl.tiles_per_split = splits > 1 ? (max_tiles + splits - 1) / splits : 0x3fffffff;
    };
    if (flags & FA_FLAG_SERIAL_KERNEL) {
        pl.kernel = kPlanSerial;
        return pl;
    }
    // Few queries per sequence and several query heads per K/V head (decoding with grouped-query
    // attention): the heads of a group share the CTA's query tile, h heads of Sq rows each with
    // h the largest divisor of the group size that fits, and every K/V tile is read and
    // multiplied once for all of them.  Only the stream kernel has this mode.
    // (Packed batches: Sq is the longest query of the batch and there is no split.)
    if (!(flags & (FA_FLAG_NO_STREAM_KERNEL | FA_FLAG_NO_HEAD_PACKING)) && Sq <= fa::kTileM / 2 &&
        Hq / Hkv >= 2) {
        const int group = Hq / Hkv;
        int hp = 1;
        for (int c = 2; c <= group && c * Sq <= fa::kTileM; ++c)
            if (group % c == 0) hp = c;
        if (hp > 1) {
            pl.kernel = kPlanStream;
            pl.pack_heads = hp;
            // (packed batches: Sk is the mean K/V length; every CTA cuts its own sequence into the C shares)
            with_splits(choose_kv_splits(num_sms, kv_splits_cfg, scratch_bytes, B, Hq, Sq, Sk, dv, causal, n_q_tiles, true, hp));
            return pl;
        }
    }
    // packed batches: no split (the lengths that decide it are on the device)
    const int pair_splits = varlen ? 1 : choose_kv_splits(num_sms, kv_splits_cfg, scratch_bytes, B, Hq, Sq, Sk, dv, causal, n_q_tiles);
    // The persistent kernel wins where a CTA's fixed cost is a visible share of an item's time and every SM gets
    // several items.  Measured on B200 against the one-item-per-CTA kernels (an A/B over item lengths,
    // `bench.py --plan-ab`): at d = 128, where both are built on the loop of fa_fwd_pair.cuh, it is 35 / 26 / 11 / 9 /
    // 7 / 3 % faster on items of 1 / 2 / 4 / 8 / 16 / 32 K/V tiles, 2 % at 64 and level at 128 and beyond; at d = 64,
    // where the per-item kernel keeps P in TMEM columns of its own, it is 5-12 % faster up to 8-tile items, level
    // at 16 and 4-5 % slower at 32; and it is a few per cent slower below two items per SM (its one-time set-up
    // and the coarser balance of a short list).  d = 192 has no room for its staging buffer.
    const long long n_items = static_cast<long long>((n_q_tiles + 1) / 2) * Hq * B;
    // (packed batches: the list has an item for every tile of the longest sequence, which Sq is;
    //  the sequences a tile does not exist in pass through the kernel's item ring empty)
    const int longest = fa::kv_tiles_for_q_tile((n_q_tiles - 1) * fa::kTileM, fa::kTileM, Sq, (varlen && Sk < Sq) ? Sq : Sk, causal);
    const bool persistent_ok = pair_splits == 1 && dqk != 192;
    bool persistent = persistent_ok && n_items >= 3ll * num_sms && longest <= (dqk == 64 ? 16 : 128);
    if (flags & FA_FLAG_NO_PERSISTENT) persistent = false;
    if ((flags & FA_FLAG_FORCE_PERSISTENT) && persistent_ok) persistent = true;
    // One query tile per CTA (twice the CTAs, each with a shorter chain) wins where the pair
    // kernel's grid does not fill the GPU or its longest CTA dominates: decided from the two
    // estimates, with a margin, each side with its own split count.
    // Causal grouped-query attention: pairing the same query tile of two heads of a group gives both
    // tiles of a pair-kernel CTA the same number of K/V tiles (no round that one of them runs alone).
    // (Without a mask it only matters for an odd number of query tiles, whose last tile would be alone.)
    // (Packed batches: every sequence's tiles pair up the same way; n_q_tiles is the longest one's.)
    const bool head_pair_ok = (causal || (n_q_tiles & 1)) && pair_splits == 1 && (Hq / Hkv) % 2 == 0 &&
                              !(flags & FA_FLAG_NO_HEAD_PACKING);
    bool stream = false;
    int stream_splits = 1;
    if (!(flags & FA_FLAG_NO_STREAM_KERNEL)) {
        // packed batches split only with a single query tile per sequence (decode-like), by the mean K/V length
        if (!varlen || n_q_tiles == 1) stream_splits = choose_kv_splits(num_sms, kv_splits_cfg, scratch_bytes, B, Hq, Sq, Sk, dv, causal, n_q_tiles, true);
        if (flags & FA_FLAG_STREAM_KERNEL) {
            stream = true;
        } else if (varlen) {
            // no estimate without the lengths: 192/128 is always ahead, and with a single query tile
            // per sequence the pair kernel's second tile would be empty, unless it is the same tile
            // of the next head of the group: with more items than SMs that halves the number of
            // CTAs and their fixed cost (B64 x 128 tokens, Hq 32 / Hkv 8: 57 vs 114 us)
            const bool paired_single_tiles = n_q_tiles == 1 && head_pair_ok && dqk != 192 && stream_splits == 1 &&
                                             static_cast<long long>(B) * Hq > num_sms;
            stream = (dqk == 192) || (n_q_tiles == 1 && !paired_single_tiles && !persistent);
        } else if (!persistent) {
            const TilingEstimate e = estimate_tilings(num_sms, B, Hq, Sq, Sk, dqk, causal, n_q_tiles, pair_splits, stream_splits, head_pair_ok);
            pl.pair_us = e.pair_us;
            pl.stream_us = e.stream_us;
            stream = e.stream_us < 0.9 * e.pair_us;
            // at d = 64 the stream kernel is also ahead on long items, closer than the estimate can
            // tell: 10 % without a mask (64 K/V tiles per query tile), 3-4 % under a causal mask from
            // 256 tiles on; with shorter causal items the pair kernel is 2-9 % ahead
            if (dqk == 64 && longest >= (causal ? 192 : 32) && pair_splits == 1 && stream_splits == 1) stream = true;
        }
    }
    // Pairs of CTAs with two-CTA MMAs (fa_fwd_duo.cuh): fixed-length launches without split-KV at head sizes
    // 128 and 192/128.
    const bool duo_ok = !varlen && dqk != 64 && pair_splits == 1 && stream_splits == 1;
    bool duo = false;
    if ((flags & FA_FLAG_TWO_CTA_KERNEL) && duo_ok) duo = true;
    if ((flags & FA_FLAG_QUAD_KERNEL) && duo_ok) {
        pl.kernel = kPlanQuad;
        const int gqa = Hq / Hkv;
        pl.quad_mode = (flags & FA_FLAG_NO_HEAD_PACKING) ? 0 : (gqa % 4 == 0 ? 2 : (gqa % 2 == 0 ? 1 : 0));
    } else if (duo) {
        pl.kernel = kPlanDuo;
        pl.head_pair = head_pair_ok;
    } else if (stream && !varlen && stream_splits == 1 && !(flags & FA_FLAG_NO_PERSISTENT) &&
               ((static_cast<long long>(n_q_tiles) * Hq * B >= 3ll * num_sms && longest <= 32) ||
                (flags & FA_FLAG_FORCE_PERSISTENT))) {
        // Many short one-tile items per SM: the stream kernel's persistent form (a CTA's fixed cost once per SM, the
        // next item's loads and first scores under the current item's tail).  Measured on B200 at 192/128 against the
        // one-item stream kernel: +18 % on items of 8 K/V tiles (no mask), +10 % on causal items of up to 16, +4.5 %
        // up to 24, +2.6 % up to 32 (config 4), within 1 % on longer items.
        pl.kernel = kPlanStreamPersistent;
    } else if (stream) {
        pl.kernel = kPlanStream;
        with_splits(stream_splits);
    } else if (persistent) {
        pl.kernel = kPlanPersistent;
        pl.head_pair = head_pair_ok;
    } else {
        pl.kernel = kPlanPair;
        with_splits(pair_splits);
        pl.head_pair = head_pair_ok;
    }
    return pl;
}

// Fills the launch parameters and starts the kernel(s); the tensor maps are ready.
// cu_q == nullptr: fixed lengths Sq, Sk.  Otherwise a packed variable-length batch whose longest
// query is Sq rows and whose sequences have about Sk keys (L2 grouping only).
fa_status run_forward(fa_handle* h, const CUtensorMap& map_q, const CUtensorMap& map_k, const CUtensorMap& map_v,
                      const CUtensorMap& map_o, void* O, float* lse, int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv, int causal,
                      float scale, const int64_t* o_strides, const int* cu_q, const int* cu_k, int total_q,
                      const LaunchPlan& pl, cudaStream_t st) {
    if (scale == 0.f) scale = 1.f / sqrtf(static_cast<float>(dqk));
    fa::FwdParams p;
    p.O = static_cast<__nv_bfloat16*>(O);
    p.o_stride_b = o_strides[0];
    p.o_stride_h = o_strides[1];
    p.o_stride_s = o_strides[2];
    p.cu_q = cu_q;
    p.cu_k = cu_k;
    p.total_q = total_q;
    p.lse = lse;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.Sq = Sq; p.Sk = Sk;
    p.causal = causal ? 1 : 0;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.n_q_tiles = (Sq + fa::kTileM - 1) / fa::kTileM;
    p.heads_per_group = heads_per_group(static_cast<long long>(Sk) * (dqk + dv) * 2, B, Hq, Hkv);
    p.sched_counter = h->sched_counter;
    p.status = h->status_dev;
    p.wait_limit_ns = h->wait_limit_ns;
    p.debug_drop_v_load = (h->flags & FA_FLAG_DEBUG_DROP_V_LOAD) ? 1 : 0;
    p.kv_splits = pl.kv_splits;
    p.tiles_per_split = pl.tiles_per_split;
    p.pack_heads = pl.pack_heads;
    p.head_pair = pl.head_pair ? 1 : 0;
    p.o_part = nullptr;
    p.lse_part = nullptr;
    if (pl.kv_splits > 1) {
        // partials [C, B*Hq, Sq, dv] and [C, B*Hq, Sq]; packed batches: [C, Hq, total_q, dv] and [C, Hq, total_q]
        const size_t rows = cu_q ? static_cast<size_t>(Hq) * total_q : static_cast<size_t>(B) * Hq * Sq;
        p.o_part = static_cast<float*>(h->scratch);
        p.lse_part = p.o_part + static_cast<size_t>(pl.kv_splits) * rows * dv;
    }
    h->last_splits = p.kv_splits;
#ifdef FA_TRACE
    p.trace = h->trace;
#endif

    if (pl.kernel == kPlanStream) {
        h->last_kernel = "fa_fwd_stream";
        if (pl.pack_heads > 1 && cu_q) {
            if (dqk == 64) return launch_stream<64, 64, true, true>(h, map_q, map_k, map_v, map_o, p, st);
            if (dqk == 128) return launch_stream<128, 128, true, true>(h, map_q, map_k, map_v, map_o, p, st);
            return launch_stream<192, 128, true, true>(h, map_q, map_k, map_v, map_o, p, st);
        }
        if (pl.pack_heads > 1) {
            if (dqk == 64) return launch_stream<64, 64, false, true>(h, map_q, map_k, map_v, map_o, p, st);
            if (dqk == 128) return launch_stream<128, 128, false, true>(h, map_q, map_k, map_v, map_o, p, st);
            return launch_stream<192, 128, false, true>(h, map_q, map_k, map_v, map_o, p, st);
        }
        if (cu_q) {
            if (dqk == 64) return launch_stream<64, 64, true>(h, map_q, map_k, map_v, map_o, p, st);
            if (dqk == 128) return launch_stream<128, 128, true>(h, map_q, map_k, map_v, map_o, p, st);
            return launch_stream<192, 128, true>(h, map_q, map_k, map_v, map_o, p, st);
        }
        if (dqk == 64) return launch_stream<64, 64>(h, map_q, map_k, map_v, map_o, p, st);
        if (dqk == 128) return launch_stream<128, 128>(h, map_q, map_k, map_v, map_o, p, st);
        return launch_stream<192, 128>(h, map_q, map_k, map_v, map_o, p, st);
    }
    if (pl.kernel == kPlanPersistent) {
        h->last_kernel = "fa_fwd_persistent";
        if (cu_q) {
            if (dqk == 64) return launch_persistent<64, 64, true>(h, map_q, map_k, map_v, map_o, p, st);
            return launch_persistent<128, 128, true>(h, map_q, map_k, map_v, map_o, p, st);
        }
        if (dqk == 64) return launch_persistent<64, 64>(h, map_q, map_k, map_v, map_o, p, st);
        return launch_persistent<128, 128>(h, map_q, map_k, map_v, map_o, p, st);
    }
    if (pl.kernel == kPlanPair) {
        h->last_kernel = "fa_fwd_pipelined";
        if (cu_q && pl.head_pair) {
            if (dqk == 64) return launch_pipelined<64, 64, true, true>(h, map_q, map_k, map_v, map_o, p, st);
            if (dqk == 128) return launch_pipelined<128, 128, true, true>(h, map_q, map_k, map_v, map_o, p, st);
            return launch_pipelined<192, 128, true, true>(h, map_q, map_k, map_v, map_o, p, st);
        }
        if (cu_q) {
            if (dqk == 64) return launch_pipelined<64, 64, true>(h, map_q, map_k, map_v, map_o, p, st);
            if (dqk == 128) return launch_pipelined<128, 128, true>(h, map_q, map_k, map_v, map_o, p, st);
            return launch_pipelined<192, 128, true>(h, map_q, map_k, map_v, map_o, p, st);
        }
        if (pl.head_pair) {
            if (dqk == 64) return launch_pipelined<64, 64, false, true>(h, map_q, map_k, map_v, map_o, p, st);
            if (dqk == 128) return launch_pipelined<128, 128, false, true>(h, map_q, map_k, map_v, map_o, p, st);
            return launch_pipelined<192, 128, false, true>(h, map_q, map_k, map_v, map_o, p, st);
        }
        if (dqk == 64) return launch_pipelined<64, 64, false>(h, map_q, map_k, map_v, map_o, p, st);
        if (dqk == 128) return launch_pipelined<128, 128, false>(h, map_q, map_k, map_v, map_o, p, st);
        return launch_pipelined<192, 128, false>(h, map_q, map_k, map_v, map_o, p, st);
    }
    if (pl.kernel == kPlanStreamPersistent) {
        h->last_kernel = "fa_fwd_stream_persistent";
        if (dqk == 64) return launch_stream_persistent<64, 64>(h, map_q, map_k, map_v, map_o, p, st);
        if (dqk == 128) return launch_stream_persistent<128, 128>(h, map_q, map_k, map_v, map_o, p, st);
        return launch_stream_persistent<192, 128>(h, map_q, map_k, map_v, map_o, p, st);
    }
    if (pl.kernel == kPlanQuad) {
        h->last_kernel = "fa_fwd_quad";
        if (dqk == 128) {
            if (pl.quad_mode == 2) return launch_quad<128, 128, 2>(h, map_q, map_k, map_v, map_o, p, st);
            if (pl.quad_mode == 1) return launch_quad<128, 128, 1>(h, map_q, map_k, map_v, map_o, p, st);
            return launch_quad<128, 128, 0>(h, map_q, map_k, map_v, map_o, p, st);
        }
        if (pl.quad_mode == 2) return launch_quad<192, 128, 2>(h, map_q, map_k, map_v, map_o, p, st);
        if (pl.quad_mode == 1) return launch_quad<192, 128, 1>(h, map_q, map_k, map_v, map_o, p, st);
        return launch_quad<192, 128, 0>(h, map_q, map_k, map_v, map_o, p, st);
    }
    if (pl.kernel == kPlanDuo) {
        h->last_kernel = "fa_fwd_duo";
        if (pl.head_pair) {
            if (dqk == 128) return launch_duo<128, 128, true>(h, map_q, map_k, map_v, map_o, p, st);
            return launch_duo<192, 128, true>(h, map_q, map_k, map_v, map_o, p, st);
        }
        if (dqk == 128) return launch_duo<128, 128, false>(h, map_q, map_k, map_v, map_o, p, st);
        return launch_duo<192, 128, false>(h, map_q, map_k, map_v, map_o, p, st);
    }
    h->last_kernel = "fa_fwd_simple";
    if (dqk == 64) return launch_simple<64, 64>(h, map_q, map_k, map_v, p, st);
    if (dqk == 128) return launch_simple<128, 128>(h, map_q, map_k, map_v, p, st);
    return launch_simple<192, 128>(h, map_q, map_k, map_v, p, st);
}

}  // namespace

extern "C" {

const char* fa_strerror(fa_status s) {
    switch (s) {
        case FA_OK: return "success";
        case FA_ERR_INVALID_ARG: return "invalid argument";
        case FA_ERR_UNSUPPORTED: return "unsupported head sizes or extents";
        case FA_ERR_CUDA: return "CUDA call failed";
        case FA_ERR_DEVICE_TIMEOUT: return "device-side wait ran out";
        case FA_ERR_NO_DEVICE: return "no usable CUDA device (need compute capability 10.x)";
        case FA_ERR_OOM: return "out of memory";
    }
    return "unknown status";
}

fa_status fa_create(fa_handle** out, const fa_config* cfg) {
    if (!out) return FA_ERR_INVALID_ARG;
    *out = nullptr;
    int device = -1;
    uint32_t flags = 0, limit_ms = 0;
    uint32_t kv_splits_cfg = 0;
    uint64_t scratch_bytes = 0;
    if (cfg) {
        // versioned by struct_size: the first four fields are mandatory, later ones optional
        if (cfg->struct_size < 16 || cfg->struct_size > sizeof(fa_config)) return FA_ERR_INVALID_ARG;
        device = cfg->device;
        flags = cfg->flags;
        limit_ms = cfg->wait_limit_ms;
        if (cfg->struct_size >= 20) kv_splits_cfg = cfg->kv_splits;
        if (cfg->struct_size >= sizeof(fa_config)) scratch_bytes = cfg->scratch_bytes;
        if (flags & ~(FA_FLAG_SERIAL_KERNEL | FA_FLAG_DEBUG_DROP_V_LOAD | FA_FLAG_NO_DEPENDENT_LAUNCH |
                      FA_FLAG_NO_PERSISTENT | FA_FLAG_FORCE_PERSISTENT | FA_FLAG_STREAM_KERNEL |
                      FA_FLAG_NO_STREAM_KERNEL | FA_FLAG_NO_HEAD_PACKING | FA_FLAG_LEGACY_PAIR_KERNEL |
                      FA_FLAG_TWO_CTA_KERNEL | FA_FLAG_QUAD_KERNEL)) return FA_ERR_INVALID_ARG;
        if (kv_splits_cfg > 256) return FA_ERR_INVALID_ARG;
    }
    if (scratch_bytes == 0) scratch_bytes = 32ull << 20;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || count <= 0) {
        cudaGetLastError();
        return FA_ERR_NO_DEVICE;
    }
    if (device < 0) {
        if (cudaGetDevice(&device) != cudaSuccess) return FA_ERR_NO_DEVICE;
    }
    if (device >= count) return FA_ERR_INVALID_ARG;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess)
        return FA_ERR_CUDA;
    if (major != 10) return FA_ERR_NO_DEVICE;
    int num_sms = 0;
    if (cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || num_sms <= 0)
        return FA_ERR_CUDA;

    fa_handle* h = new (std::nothrow) fa_handle();
    if (!h) return FA_ERR_OOM;
    h->device = device;
    h->num_sms = num_sms;
    h->flags = flags;
    h->kv_splits_cfg = kv_splits_cfg;
    if (limit_ms) h->wait_limit_ns = static_cast<unsigned long long>(limit_ms) * 1000000ull;
    h->maps.reserve(kMapCacheSize);

    DeviceGuard guard(device);
    if (!guard.ok()) { delete h; return FA_ERR_CUDA; }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaGetLastError();
        delete h;
        return FA_ERR_CUDA;
    }
    h->encode = reinterpret_cast<EncodeTiledFn>(fn);
    if (cudaHostAlloc(reinterpret_cast<void**>(&h->status_host), 16, cudaHostAllocMapped) != cudaSuccess) {
        cudaGetLastError();
        delete h;
        return FA_ERR_OOM;
    }
    memset(h->status_host, 0, 16);
    if (cudaHostGetDevicePointer(reinterpret_cast<void**>(&h->status_dev), h->status_host, 0) != cudaSuccess) {
        cudaGetLastError();
        cudaFreeHost(h->status_host);
        delete h;
        return FA_ERR_CUDA;
    }
    if (cudaMalloc(&h->scratch, scratch_bytes) != cudaSuccess) {
        cudaGetLastError();
        cudaFreeHost(h->status_host);
        delete h;
        return FA_ERR_OOM;
    }
    h->scratch_bytes = scratch_bytes;
    if (cudaMalloc(reinterpret_cast<void**>(&h->sched_counter), 256) != cudaSuccess ||
        cudaMemset(h->sched_counter, 0, 256) != cudaSuccess) {
        cudaGetLastError();
        if (h->sched_counter) cudaFree(h->sched_counter);
        cudaFree(h->scratch);
        cudaFreeHost(h->status_host);
        delete h;
        return FA_ERR_OOM;
    }
    *out = h;
    return FA_OK;
}

fa_status fa_destroy(fa_handle* h) {
    if (!h) return FA_OK;
    DeviceGuard guard(h->device);
    fa_status s = FA_OK;
    for (int i = 0; i < 5; ++i)
        if (h->stage[i] && cudaFree(h->stage[i]) != cudaSuccess) s = FA_ERR_CUDA;
    for (cudaEvent_t e : h->ev_in) if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : h->ev_done) if (e) cudaEventDestroy(e);
    if (h->ev_start) cudaEventDestroy(h->ev_start);
    if (h->ev_out_done) cudaEventDestroy(h->ev_out_done);
    if (h->copy_in) cudaStreamDestroy(h->copy_in);
    if (h->copy_out) cudaStreamDestroy(h->copy_out);
    if (h->scratch && cudaFree(h->scratch) != cudaSuccess) s = FA_ERR_CUDA;
    if (h->sched_counter && cudaFree(h->sched_counter) != cudaSuccess) s = FA_ERR_CUDA;
    if (h->status_host && cudaFreeHost(h->status_host) != cudaSuccess) s = FA_ERR_CUDA;
    delete h;
    return s;
}

fa_status fa_last_status(fa_handle* h, uint32_t* detail) {
    if (!h) return FA_ERR_INVALID_ARG;
    volatile uint32_t* sw = h->status_host;
    const uint32_t code = sw[0];
    const uint32_t who = sw[1];
    if (detail) *detail = code ? who : 0u;
    if (code) {
        sw[0] = 0;
        sw[1] = 0;
        // A persistent launch that gave up has not made all of its draws from the ticket counter, which the last
        // draw of a complete launch puts back to zero: zero it here, or the next persistent launch would start in the
        // middle of its item list.  (The caller synchronised before asking, so no launch is using the counter.)
        if (h->sched_counter) {
            DeviceGuard guard(h->device);
            if (guard.ok()) cudaMemset(h->sched_counter, 0, sizeof(unsigned int));
        }
    }
    return code == 0 ? FA_OK : (code == FA_ERR_DEVICE_TIMEOUT ? FA_ERR_DEVICE_TIMEOUT : FA_ERR_CUDA);
}

fa_status fa_debug_set_drop_v_load(fa_handle* h, int enabled) {
    if (!h) return FA_ERR_INVALID_ARG;
    if (enabled) h->flags |= FA_FLAG_DEBUG_DROP_V_LOAD;
    else h->flags &= ~FA_FLAG_DEBUG_DROP_V_LOAD;
    return FA_OK;
}

uint64_t fa_launch_count(const fa_handle* h) { return h ? h->launches : 0; }
int fa_last_kv_splits(const fa_handle* h) { return h ? h->last_splits : 0; }
const char* fa_last_kernel_name(const fa_handle* h) { return h ? h->last_kernel : ""; }

fa_status fa_forward_strided(fa_handle* h, const void* Q, const void* K, const void* V, void* O, float* lse,
                             int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv, int causal,
                             float scale, const int64_t* q_strides, const int64_t* k_strides,
                             const int64_t* v_strides, const int64_t* o_strides, void* stream) {
    if (!h) return FA_ERR_INVALID_ARG;
    fa_status s = check_args(Q, K, V, O, lse, B, Hq, Hkv, Sq, Sk, dqk, dv, scale, true);
    if (s != FA_OK) return s;
    if (!q_strides || !k_strides || !v_strides || !o_strides) return FA_ERR_INVALID_ARG;
    for (int i = 0; i < 3; ++i) {
        // TMA wants every stride to be a multiple of 16 bytes; 16-byte row stores want the same of O
        if (q_strides[i] <= 0 || k_strides[i] <= 0 || v_strides[i] <= 0 || o_strides[i] <= 0) return FA_ERR_INVALID_ARG;
        if ((q_strides[i] | k_strides[i] | v_strides[i] | o_strides[i]) & 7) return FA_ERR_INVALID_ARG;
    }
    if (q_strides[2] < dqk || k_strides[2] < dqk || v_strides[2] < dv || o_strides[2] < dv) return FA_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok()) return FA_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const CUtensorMap *mq = nullptr, *mk = nullptr, *mv = nullptr, *mo = nullptr;
    const LaunchPlan pl = plan_launch(h->num_sms, h->flags, h->kv_splits_cfg, h->scratch_bytes, false,
                                      B, Hq, Hkv, Sq, Sk, dqk, dv, causal ? 1 : 0);
    // packed heads: the box of Q and O is the Sq rows of pack_heads heads
    const int q_box_rows = pl.pack_heads > 1 ? Sq : fa::kTileM;
    if ((s = get_map(h, Q, dqk, Sq, Hq, B, q_strides[0], q_strides[1], q_strides[2], q_box_rows, &mq, 2, pl.pack_heads)) != FA_OK) return s;
    CUtensorMap map_q = *mq;   // copies: a later insertion may evict or move cache entries
    // (the two-CTA kernel loads K in boxes of 64 keys: each CTA of a pair keeps half of a K tile)
    const int k_box_rows = (pl.kernel == kPlanDuo || pl.kernel == kPlanQuad) ? fa::kTileN / 2 : fa::kTileN;
    if ((s = get_map(h, K, dqk, Sk, Hkv, B, k_strides[0], k_strides[1], k_strides[2], k_box_rows, &mk)) != FA_OK) return s;
    CUtensorMap map_k = *mk;
    if ((s = get_map(h, V, dv, Sk, Hkv, B, v_strides[0], v_strides[1], v_strides[2], fa::kTileN, &mv)) != FA_OK) return s;
    CUtensorMap map_v = *mv;
    if ((s = get_map(h, O, dv, Sq, Hq, B, o_strides[0], o_strides[1], o_strides[2], q_box_rows, &mo, 2, pl.pack_heads)) != FA_OK) return s;
    CUtensorMap map_o = *mo;

    return run_forward(h, map_q, map_k, map_v, map_o, O, lse, B, Hq, Hkv, Sq, Sk, dqk, dv, causal, scale, o_strides,
                       nullptr, nullptr, 0, pl, st);
}

fa_status fa_forward(fa_handle* h, const void* Q, const void* K, const void* V, void* O, float* lse,
                     int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv, int causal,
                     float scale, void* stream) {
    // contiguous [B, H, S, d]
    const int64_t qs[3] = {static_cast<int64_t>(Hq) * Sq * dqk, static_cast<int64_t>(Sq) * dqk, dqk};
    const int64_t ks[3] = {static_cast<int64_t>(Hkv) * Sk * dqk, static_cast<int64_t>(Sk) * dqk, dqk};
    const int64_t vs[3] = {static_cast<int64_t>(Hkv) * Sk * dv, static_cast<int64_t>(Sk) * dv, dv};
    const int64_t os[3] = {static_cast<int64_t>(Hq) * Sq * dv, static_cast<int64_t>(Sq) * dv, dv};
    return fa_forward_strided(h, Q, K, V, O, lse, B, Hq, Hkv, Sq, Sk, dqk, dv, causal, scale, qs, ks, vs, os, stream);
}

fa_status fa_forward_varlen(fa_handle* h, const void* Q, const void* K, const void* V, void* O, float* lse,
                            const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k, int B, int total_q,
                            int total_k, int max_sq, int Hq, int Hkv, int dqk, int dv, int causal, float scale,
                            void* stream) {
    if (!h || !cu_seqlens_q || !cu_seqlens_k) return FA_ERR_INVALID_ARG;
    if (B < 0 || total_q < 0 || total_k < 0 || max_sq < 0 || max_sq > total_q) return FA_ERR_INVALID_ARG;
    if (misaligned(cu_seqlens_q, 4) || misaligned(cu_seqlens_k, 4)) return FA_ERR_INVALID_ARG;
    if (B == 0 || total_q == 0 || max_sq == 0) return FA_OK;           // no query rows: nothing to write
    // K and V may be empty (every row then gets O = 0, lse = -inf); the maps still need one row
    fa_status s = check_args(Q, K, V, O, lse, B, Hq, Hkv, max_sq, total_k > 0 ? total_k : 1, dqk, dv, scale, true);
    if (s != FA_OK) return s;
    DeviceGuard guard(h->device);
    if (!guard.ok()) return FA_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // packed [total, H, d]: one batch slice, rows H*d apart, heads d apart
    const int mean_sk = (total_k + B - 1) / B > 0 ? (total_k + B - 1) / B : 1;
    const LaunchPlan pl = plan_launch(h->num_sms, h->flags, h->kv_splits_cfg, h->scratch_bytes, true,
                                      B, Hq, Hkv, max_sq, mean_sk, dqk, dv, causal ? 1 : 0);
    // packed heads: the box of Q is the max_sq rows (from the sequence's first row) of pack_heads heads
    const int q_box_rows = pl.pack_heads > 1 ? max_sq : fa::kTileM;
    const CUtensorMap *mq = nullptr, *mk = nullptr, *mv = nullptr, *mo = nullptr;
    const int rows_k = total_k > 0 ? total_k : 1;   // an empty K/V still gets a valid map; no tile of it is ever read
    if ((s = get_map(h, Q, dqk, total_q, Hq, 1, static_cast<long long>(total_q) * Hq * dqk, dqk,
                     static_cast<long long>(Hq) * dqk, q_box_rows, &mq, 2, pl.pack_heads)) != FA_OK) return s;
    CUtensorMap map_q = *mq;
    if ((s = get_map(h, K, dqk, rows_k, Hkv, 1, static_cast<long long>(rows_k) * Hkv * dqk, dqk,
                     static_cast<long long>(Hkv) * dqk, fa::kTileN, &mk)) != FA_OK) return s;
    CUtensorMap map_k = *mk;
    if ((s = get_map(h, V, dv, rows_k, Hkv, 1, static_cast<long long>(rows_k) * Hkv * dv, dv,
                     static_cast<long long>(Hkv) * dv, fa::kTileN, &mv)) != FA_OK) return s;
    CUtensorMap map_v = *mv;
    if ((s = get_map(h, O, dv, total_q, Hq, 1, static_cast<long long>(total_q) * Hq * dv, dv,
                     static_cast<long long>(Hq) * dv, fa::kTileM, &mo)) != FA_OK) return s;
    CUtensorMap map_o = *mo;
    const int64_t os[3] = {0, dv, static_cast<int64_t>(Hq) * dv};
    return run_forward(h, map_q, map_k, map_v, map_o, O, lse, B, Hq, Hkv, max_sq, mean_sk, dqk, dv, causal, scale, os,
                       cu_seqlens_q, cu_seqlens_k, total_q, pl, st);
}

// Both 8-bit entry points: fp32 scales per 128-row block (q_scale, k_scale, v_scale; each may be NULL), or, with
// q_sf != NULL, the MX form with e8m0 scale atoms (q_sf, k_sf, v_sf).
static fa_status forward_fp8_common(fa_handle* h, const void* Q8, const void* K8, const void* V8,
                                    const float* q_scale, const float* k_scale, const float* v_scale,
                                    const uint8_t* q_sf, const uint8_t* k_sf, const uint8_t* v_sf,
                                    void* O, float* lse, int B, int Hq, int Hkv, int Sq, int Sk, int d, int causal,
                                    float scale, void* stream) {
    if (!h) return FA_ERR_INVALID_ARG;
    const bool mx = q_sf != nullptr;
    // d = 192: the 192/128 shapes (Q and K of head size 192, V and O of 128); fp32 block scales only
    if (d != 64 && d != 128 && !(d == 192 && !mx)) return (d > 0) ? FA_ERR_UNSUPPORTED : FA_ERR_INVALID_ARG;
    const int dv = (d == 192) ? 128 : d;
    fa_status s = check_args(Q8, K8, V8, O, lse, B, Hq, Hkv, Sq, Sk, d, dv, scale, true);
    if (s != FA_OK) return s;
    if ((q_scale && misaligned(q_scale, 4)) || (k_scale && misaligned(k_scale, 4)) || (v_scale && misaligned(v_scale, 4)))
        return FA_ERR_INVALID_ARG;
    if (mx && (!k_sf || !v_sf || misaligned(q_sf, 16) || misaligned(k_sf, 16) || misaligned(v_sf, 16))) return FA_ERR_INVALID_ARG;
    if (h->flags & FA_FLAG_SERIAL_KERNEL) return FA_ERR_UNSUPPORTED;
    DeviceGuard guard(h->device);
    if (!guard.ok()) return FA_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (scale == 0.f) scale = 1.f / sqrtf(static_cast<float>(d));

    // The tiling is planned as for 16-bit operands of the same shape (the 8-bit kernels' per-CTA
    // costs are lower by a similar factor in both tilings).  Only the stream tiling splits K/V
    // and packs heads.
    // (The MX form runs on the stream tiling with one head per query tile: its scale atoms follow the tile's rows.)
    // (So does head size 192/128: only the stream kernel has it.)
    const uint32_t plan_flags = (mx || d == 192) ? ((h->flags & ~(FA_FLAG_NO_STREAM_KERNEL | FA_FLAG_FORCE_PERSISTENT | FA_FLAG_TWO_CTA_KERNEL)) |
                                                    FA_FLAG_STREAM_KERNEL | FA_FLAG_NO_HEAD_PACKING)
                                                 : h->flags;
    LaunchPlan pl = plan_launch(h->num_sms, plan_flags, h->kv_splits_cfg, h->scratch_bytes, false,
                                B, Hq, Hkv, Sq, Sk, d, dv, causal ? 1 : 0);
    if (pl.kernel == kPlanStreamPersistent) pl.kernel = kPlanStream;      // (the 8-bit stream kernel has no persistent form)
    const int q_box_rows = pl.pack_heads > 1 ? Sq : fa::kTileM;
    // an e4m3 row is d bytes: one box column of d bytes, swizzled over d bytes
    const CUtensorMap *mq = nullptr, *mk = nullptr, *mv = nullptr, *mo = nullptr;
    const long long hq_stride = static_cast<long long>(Sq) * d, hk_stride = static_cast<long long>(Sk) * d;
    const long long ho_stride = static_cast<long long>(Sq) * dv, hv_stride = static_cast<long long>(Sk) * dv;
    // (a row of 192 bytes is loaded as two boxes: 128 bytes with the 128-byte swizzle, 64 bytes with the 64-byte one)
    const int sw_qk = (d == 64) ? 64 : 128;
    if ((s = get_map(h, Q8, d, Sq, Hq, B, hq_stride * Hq, hq_stride, d, q_box_rows, &mq, 1, pl.pack_heads, sw_qk)) != FA_OK) return s;
    CUtensorMap map_q = *mq;
    if ((s = get_map(h, K8, d, Sk, Hkv, B, hk_stride * Hkv, hk_stride, d, fa::kTileN, &mk, 1, 1, sw_qk)) != FA_OK) return s;
    CUtensorMap map_k = *mk;
    if ((s = get_map(h, V8, dv, Sk, Hkv, B, hv_stride * Hkv, hv_stride, dv, fa::kTileN, &mv, 1, 1, dv)) != FA_OK) return s;
    CUtensorMap map_v = *mv;
    if ((s = get_map(h, O, dv, Sq, Hq, B, ho_stride * Hq, ho_stride, dv, q_box_rows, &mo, 2, pl.pack_heads)) != FA_OK) return s;
    CUtensorMap map_o = *mo;
    CUtensorMap map_q2 = map_q, map_k2 = map_k;
    if (d == 192) {
        if ((s = get_map(h, Q8, d, Sq, Hq, B, hq_stride * Hq, hq_stride, d, q_box_rows, &mq, 1, 1, 64)) != FA_OK) return s;
        map_q2 = *mq;
        if ((s = get_map(h, K8, d, Sk, Hkv, B, hk_stride * Hkv, hk_stride, d, fa::kTileN, &mk, 1, 1, 64)) != FA_OK) return s;
        map_k2 = *mk;
    }

    fa::FwdParams p;
    memset(&p, 0, sizeof p);
    p.O = static_cast<__nv_bfloat16*>(O);
    p.o_stride_b = ho_stride * Hq;
    p.o_stride_h = ho_stride;
    p.o_stride_s = dv;
    p.lse = lse;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.Sq = Sq; p.Sk = Sk;
    p.causal = causal ? 1 : 0;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.n_q_tiles = (Sq + fa::kTileM - 1) / fa::kTileM;
    p.heads_per_group = heads_per_group(static_cast<long long>(Sk) * (d + dv), B, Hq, Hkv);      // one byte per element
    p.status = h->status_dev;
    p.wait_limit_ns = h->wait_limit_ns;
    p.debug_drop_v_load = (h->flags & FA_FLAG_DEBUG_DROP_V_LOAD) ? 1 : 0;
    fa::Fp8Params f;
    f.q_scale = q_scale; f.k_scale = k_scale; f.v_scale = v_scale;
    f.q_sf = q_sf; f.k_sf = k_sf; f.v_sf = v_sf;
    f.n_kv_tiles = (Sk + fa::kTileN - 1) / fa::kTileN;
    const bool use_stream = pl.kernel == kPlanStream;
    p.kv_splits = use_stream ? pl.kv_splits : 1;
    p.tiles_per_split = use_stream ? pl.tiles_per_split : 0x3fffffff;
    p.pack_heads = pl.pack_heads;
    // A pack of at most 32 (64) rows is loaded four times (twice) and every copy takes a quarter
    // (half) of each K/V tile's keys: the partials per query row multiply accordingly.
    int copies = 1;
    if (use_stream && pl.pack_heads > 1) {
        const int rows = pl.pack_heads * Sq;
        copies = rows <= 32 ? 4 : (rows <= 64 ? 2 : 1);
        // every copy is one more partial per split for the merge kernel to read: with many splits
        // (short CTAs, where the exponentials saved are few) the merge would cost more than it saves
        while (copies > 1 && copies * p.kv_splits > 32) copies /= 2;
        const unsigned long long per_partial = static_cast<unsigned long long>(B) * Hq * Sq * (dv + 1) * 4ull;
        while (copies > 1 && per_partial * p.kv_splits * copies > h->scratch_bytes) copies /= 2;
    }
    const int n_partials = p.kv_splits * copies;
    if (n_partials > 1) {
        p.o_part = static_cast<float*>(h->scratch);
        p.lse_part = p.o_part + static_cast<size_t>(n_partials) * B * Hq * Sq * dv;
    }
    h->last_splits = p.kv_splits;
    h->last_kernel = use_stream ? (mx ? "fa_fwd_mxfp8_stream" : "fa_fwd_fp8_stream") : "fa_fwd_fp8";
    if (mx && !use_stream) return FA_ERR_UNSUPPORTED;       // (cannot happen: the stream tiling was forced above)

    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(512, 1, 1);
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = (h->flags & FA_FLAG_NO_DEPENDENT_LAUNCH) ? 0 : 1;
    const bool d128 = (d == 128);
    if (use_stream) {
        const int smem = d == 192 ? fa::fp8_stream_smem_bytes<192>() : (d128 ? fa::fp8_stream_smem_bytes<128>() : fa::fp8_stream_smem_bytes<64>());
        static_assert(fa::fp8_stream_smem_bytes<128>() <= 227 * 1024 && fa::fp8_stream_smem_bytes<192>() <= 227 * 1024,
                      "shared memory budget exceeded");
        const bool pack = pl.pack_heads > 1;
        using Kernel = void (*)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, fa::FwdParams, fa::Fp8Params);
        // variant: 0 = one head per tile, 1..3 = packed heads with 1, 2, 4 copies of the rows
        const int variant = !pack ? 0 : (copies == 4 ? 3 : (copies == 2 ? 2 : 1));
        static const Kernel kernels[2][4] = {
            {fa::fa_fwd_fp8_stream_kernel<64, false, 1>, fa::fa_fwd_fp8_stream_kernel<64, true, 1>,
             fa::fa_fwd_fp8_stream_kernel<64, true, 2>, fa::fa_fwd_fp8_stream_kernel<64, true, 4>},
            {fa::fa_fwd_fp8_stream_kernel<128, false, 1>, fa::fa_fwd_fp8_stream_kernel<128, true, 1>,
             fa::fa_fwd_fp8_stream_kernel<128, true, 2>, fa::fa_fwd_fp8_stream_kernel<128, true, 4>}};
        Kernel kernel = kernels[d128 ? 1 : 0][variant];
        if (mx) kernel = d128 ? fa::fa_fwd_fp8_stream_kernel<128, false, 1, true> : fa::fa_fwd_fp8_stream_kernel<64, false, 1, true>;
        if (d == 192) kernel = fa::fa_fwd_fp8_stream_kernel<192, false, 1, false>;
        if ((s = ensure_smem_attr(h, kernel, smem)) != FA_OK) return s;
        const long long n_ctas = (pack ? static_cast<long long>(Hq / pl.pack_heads) : static_cast<long long>(p.n_q_tiles) * Hq) * B * p.kv_splits;
        if (n_ctas > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;
        cfg.gridDim = dim3(static_cast<unsigned>(n_ctas), 1, 1);
        cfg.dynamicSmemBytes = smem;
        if (cudaLaunchKernelEx(&cfg, kernel, map_q, map_k, map_v, map_o, map_q2, map_k2, p, f) != cudaSuccess) return FA_ERR_CUDA;
        h->launches += 1;
        if (n_partials > 1) {
            const long long n_rows = static_cast<long long>(B) * Hq * Sq;
            const long long blocks = (n_rows + 3) / 4;
            if (blocks > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;
            cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
            cfg.blockDim = dim3(128, 1, 1);
            cfg.dynamicSmemBytes = 0;
            auto combine = dv == 128 ? fa::fa_combine_kernel<128> : fa::fa_combine_kernel<64>;
            if (cudaLaunchKernelEx(&cfg, combine, static_cast<const float*>(p.o_part),
                                   static_cast<const float*>(p.lse_part), p.O, p.lse, n_rows, n_partials, p.Hq, p.Sq,
                                   p.o_stride_b, p.o_stride_h, p.o_stride_s) != cudaSuccess) return FA_ERR_CUDA;
            h->launches += 1;
        }
        return FA_OK;
    }
    const int smem = d128 ? fa::fp8_smem_bytes<128>() : fa::fp8_smem_bytes<64>();
    static_assert(fa::fp8_smem_bytes<128>() <= 227 * 1024, "shared memory budget exceeded");
    // causal grouped heads: the CTA's two tiles are one query tile of two adjacent heads (see plan_launch)
    const bool hp = pl.head_pair && (pl.kernel == kPlanPair || pl.kernel == kPlanPersistent);
    auto kernel = hp ? (d128 ? fa::fa_fwd_fp8_kernel<128, true> : fa::fa_fwd_fp8_kernel<64, true>)
                     : (d128 ? fa::fa_fwd_fp8_kernel<128, false> : fa::fa_fwd_fp8_kernel<64, false>);
    if ((s = ensure_smem_attr(h, kernel, smem)) != FA_OK) return s;
    const long long n_ctas = (hp ? static_cast<long long>(p.n_q_tiles) * (Hq / 2) : static_cast<long long>((p.n_q_tiles + 1) / 2) * Hq) * B;
    if (n_ctas > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;
    cfg.gridDim = dim3(static_cast<unsigned>(n_ctas), 1, 1);
    cfg.dynamicSmemBytes = smem;
    if (cudaLaunchKernelEx(&cfg, kernel, map_q, map_k, map_v, map_o, p, f) != cudaSuccess) return FA_ERR_CUDA;
    h->launches += 1;
    return FA_OK;
}

fa_status fa_forward_fp8(fa_handle* h, const void* Q8, const void* K8, const void* V8,
                         const float* q_scale, const float* k_scale, const float* v_scale,
                         void* O, float* lse, int B, int Hq, int Hkv, int Sq, int Sk, int d, int causal,
                         float scale, void* stream) {
    return forward_fp8_common(h, Q8, K8, V8, q_scale, k_scale, v_scale, nullptr, nullptr, nullptr, O, lse, B, Hq, Hkv, Sq, Sk, d,
                              causal, scale, stream);
}

fa_status fa_forward_mxfp8(fa_handle* h, const void* Q8, const void* K8, const void* V8,
                           const uint8_t* q_sf, const uint8_t* k_sf, const uint8_t* v_sf,
                           void* O, float* lse, int B, int Hq, int Hkv, int Sq, int Sk, int d, int causal,
                           float scale, void* stream) {
    if (!q_sf || !k_sf || !v_sf) return FA_ERR_INVALID_ARG;
    return forward_fp8_common(h, Q8, K8, V8, nullptr, nullptr, nullptr, q_sf, k_sf, v_sf, O, lse, B, Hq, Hkv, Sq, Sk, d,
                              causal, scale, stream);
}

fa_status fa_plan(int num_sms, const fa_config* cfg, int varlen, int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv,
                  int causal, fa_plan_info* out) {
    if (!out || num_sms <= 0 || B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || Hq % Hkv != 0) return FA_ERR_INVALID_ARG;
    const bool dims_ok = (dqk == 64 && dv == 64) || (dqk == 128 && dv == 128) || (dqk == 192 && dv == 128);
    if (!dims_ok) return FA_ERR_UNSUPPORTED;
    uint32_t flags = 0, splits_cfg = 0;
    uint64_t scratch = 32ull << 20;
    if (cfg) {
        if (cfg->struct_size < 16) return FA_ERR_INVALID_ARG;
        flags = cfg->flags;
        if (cfg->struct_size >= 20) splits_cfg = cfg->kv_splits;
        if (cfg->struct_size >= sizeof(fa_config) && cfg->scratch_bytes) scratch = cfg->scratch_bytes;
    }
    const LaunchPlan pl = plan_launch(num_sms, flags, splits_cfg, static_cast<size_t>(scratch), varlen != 0,
                                      B, Hq, Hkv, Sq, Sk, dqk, dv, causal ? 1 : 0);
    static const char* const names[7] = {"fa_fwd_simple", "fa_fwd_pipelined", "fa_fwd_persistent", "fa_fwd_stream", "fa_fwd_duo", "fa_fwd_quad",
                                         "fa_fwd_stream_persistent"};
    out->kernel = names[pl.kernel];
    // the one-item-per-CTA tiling with two query tiles has a kernel of its own at head size 128
    if (pl.kernel == kPlanPair && dqk == 128 && dv == 128 && !(flags & FA_FLAG_LEGACY_PAIR_KERNEL)) out->kernel = "fa_fwd_pair";
    out->kv_splits = pl.kv_splits;
    out->heads_per_tile = pl.pack_heads;
    const long long n_q_tiles = (Sq + fa::kTileM - 1) / fa::kTileM;
    long long ctas = 0;
    switch (pl.kernel) {
        case kPlanSerial: ctas = n_q_tiles * Hq * B; break;
        case kPlanPair: ctas = (pl.head_pair ? n_q_tiles * (Hq / 2) : ((n_q_tiles + 1) / 2) * Hq) * B * pl.kv_splits; break;
        case kPlanStreamPersistent:
            ctas = n_q_tiles * Hq * B;
            if (ctas > num_sms) ctas = num_sms;
            break;
        case kPlanQuad: {
            const int heads = pl.quad_mode == 0 ? 1 : (pl.quad_mode == 1 ? 2 : 4);
            ctas = 2 * ((n_q_tiles + 4 / heads - 1) / (4 / heads)) * (Hq / heads) * B;
            break;
        }
        case kPlanDuo: ctas = 2 * (pl.head_pair ? n_q_tiles * (Hq / 2) : ((n_q_tiles + 1) / 2) * Hq) * B; break;
        case kPlanPersistent:
            ctas = (pl.head_pair ? n_q_tiles * (Hq / 2) : ((n_q_tiles + 1) / 2) * Hq) * B;
            if (ctas > num_sms) ctas = num_sms;
            break;
        default: ctas = n_q_tiles * (Hq / pl.pack_heads) * B * pl.kv_splits; break;
    }
    out->ctas = ctas;
    out->estimate_pair_us = pl.pair_us;
    out->estimate_stream_us = pl.stream_us;
    return FA_OK;
}

fa_status fa_forward_host(fa_handle* h, const void* Qh, const void* Kh, const void* Vh, void* Oh,
                          float* lse_h, int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv,
                          int causal, float scale, void* stream) {
    if (!h) return FA_ERR_INVALID_ARG;
    fa_status s = check_args(Qh, Kh, Vh, Oh, lse_h, B, Hq, Hkv, Sq, Sk, dqk, dv, scale, false);
    if (s != FA_OK) return s;
    DeviceGuard guard(h->device);
    if (!guard.ok()) return FA_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t nq = static_cast<size_t>(B) * Hq * Sq;
    const size_t nk = static_cast<size_t>(B) * Hkv * Sk;
    const size_t bytes[5] = {nq * dqk * 2, nk * dqk * 2, nk * dv * 2, nq * dv * 2, nq * 4};
    for (int i = 0; i < 5; ++i) {
        if (h->stage_cap[i] >= bytes[i]) continue;
        if (h->stage[i]) { cudaFree(h->stage[i]); h->stage[i] = nullptr; h->stage_cap[i] = 0; }
        if (cudaMalloc(&h->stage[i], bytes[i]) != cudaSuccess) { cudaGetLastError(); return FA_ERR_OOM; }
        h->stage_cap[i] = bytes[i];
    }
    // Large problems are cut into chunks of whole (batch, K/V head) units, which are independent problems and lie
    // contiguously in all five tensors: the copy of chunk i+1 to the device and of chunk i-1 back to the host run
    // on two copy streams of the handle under the kernel of chunk i.  Small problems gain nothing from that (measured
    // on 42 MB: the pieces' copies drop to 32-35 GB/s and the launches add up), so they go through in one piece.
    const long long units = static_cast<long long>(B) * Hkv;
    const size_t total = bytes[0] + bytes[1] + bytes[2] + bytes[3] + (lse_h ? bytes[4] : 0);
    int chunks = 1;
    if (total >= (256ull << 20) && units >= 2) {
        chunks = static_cast<int>(total >> 27);          // about 128 MB of traffic per chunk
        if (chunks > 16) chunks = 16;
        if (chunks > units) chunks = static_cast<int>(units);
        if (chunks < 2) chunks = 2;
    }
    if (chunks == 1) {
        const void* src[3] = {Qh, Kh, Vh};
        for (int i = 0; i < 3; ++i)
            if (cudaMemcpyAsync(h->stage[i], src[i], bytes[i], cudaMemcpyHostToDevice, st) != cudaSuccess)
                return FA_ERR_CUDA;
        s = fa_forward(h, h->stage[0], h->stage[1], h->stage[2], h->stage[3],
                       lse_h ? static_cast<float*>(h->stage[4]) : nullptr,
                       B, Hq, Hkv, Sq, Sk, dqk, dv, causal, scale, stream);
        if (s != FA_OK) return s;
        if (cudaMemcpyAsync(Oh, h->stage[3], bytes[3], cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return FA_ERR_CUDA;
        if (lse_h && cudaMemcpyAsync(lse_h, h->stage[4], bytes[4], cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return FA_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return FA_ERR_CUDA;
        return FA_OK;
    }
    if (!h->copy_in) {
        if (cudaStreamCreateWithFlags(&h->copy_in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&h->copy_out, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&h->ev_start, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&h->ev_out_done, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            return FA_ERR_CUDA;
        }
    }
    // A chunk is either a range of K/V heads of one batch entry (with the query heads of those groups) or a range
    // of whole batch entries.
    const int group = Hq / Hkv;
    const bool by_batch = B >= chunks;
    const int per_batch = by_batch ? 1 : (chunks + B - 1) / B;             // chunks per batch entry
    const int heads_per_chunk = by_batch ? Hkv : (Hkv + per_batch - 1) / per_batch;
    const int batches_per_chunk = by_batch ? (B + chunks - 1) / chunks : 1;
    const int max_chunks = by_batch ? chunks : B * per_batch;
    while (static_cast<int>(h->ev_in.size()) < max_chunks) {
        cudaEvent_t a = nullptr, b2 = nullptr;
        if (cudaEventCreateWithFlags(&a, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&b2, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            return FA_ERR_CUDA;
        }
        h->ev_in.push_back(a);
        h->ev_done.push_back(b2);
    }
    // what the caller queued on `stream` before this call comes first
    if (cudaEventRecord(h->ev_start, st) != cudaSuccess || cudaStreamWaitEvent(h->copy_in, h->ev_start, 0) != cudaSuccess ||
        cudaStreamWaitEvent(h->copy_out, h->ev_start, 0) != cudaSuccess) return FA_ERR_CUDA;
    int n = 0;
    for (int b0 = 0; b0 < B; b0 += batches_per_chunk) {
        const int nb = (B - b0 < batches_per_chunk) ? (B - b0) : batches_per_chunk;
        for (int k0 = 0; k0 < Hkv; k0 += heads_per_chunk, ++n) {
            const int nkh = (Hkv - k0 < heads_per_chunk) ? (Hkv - k0) : heads_per_chunk;
            const int nqh = nkh * group;
            // element offsets of the chunk's first row, and its extents (whole batch entries: every head)
            const size_t q_off = (static_cast<size_t>(b0) * Hq + static_cast<size_t>(k0) * group) * Sq;
            const size_t k_off = (static_cast<size_t>(b0) * Hkv + k0) * Sk;
            const size_t q_rows = by_batch ? static_cast<size_t>(nb) * Hq * Sq : static_cast<size_t>(nqh) * Sq;
            const size_t k_rows = by_batch ? static_cast<size_t>(nb) * Hkv * Sk : static_cast<size_t>(nkh) * Sk;
            char* dq = static_cast<char*>(h->stage[0]) + q_off * dqk * 2;
            char* dk = static_cast<char*>(h->stage[1]) + k_off * dqk * 2;
            char* dvp = static_cast<char*>(h->stage[2]) + k_off * dv * 2;
            char* dop = static_cast<char*>(h->stage[3]) + q_off * dv * 2;
            float* dl = static_cast<float*>(h->stage[4]) + q_off;
            if (cudaMemcpyAsync(dq, static_cast<const char*>(Qh) + q_off * dqk * 2, q_rows * dqk * 2, cudaMemcpyHostToDevice, h->copy_in) != cudaSuccess ||
                cudaMemcpyAsync(dk, static_cast<const char*>(Kh) + k_off * dqk * 2, k_rows * dqk * 2, cudaMemcpyHostToDevice, h->copy_in) != cudaSuccess ||
                cudaMemcpyAsync(dvp, static_cast<const char*>(Vh) + k_off * dv * 2, k_rows * dv * 2, cudaMemcpyHostToDevice, h->copy_in) != cudaSuccess ||
                cudaEventRecord(h->ev_in[n], h->copy_in) != cudaSuccess || cudaStreamWaitEvent(st, h->ev_in[n], 0) != cudaSuccess)
                return FA_ERR_CUDA;
            s = fa_forward(h, dq, dk, dvp, dop, lse_h ? dl : nullptr, by_batch ? nb : 1, by_batch ? Hq : nqh, by_batch ? Hkv : nkh,
                           Sq, Sk, dqk, dv, causal, scale, stream);
            if (s != FA_OK) return s;
            if (cudaEventRecord(h->ev_done[n], st) != cudaSuccess || cudaStreamWaitEvent(h->copy_out, h->ev_done[n], 0) != cudaSuccess ||
                cudaMemcpyAsync(static_cast<char*>(Oh) + q_off * dv * 2, dop, q_rows * dv * 2, cudaMemcpyDeviceToHost, h->copy_out) != cudaSuccess)
                return FA_ERR_CUDA;
            if (lse_h && cudaMemcpyAsync(lse_h + q_off, dl, q_rows * 4, cudaMemcpyDeviceToHost, h->copy_out) != cudaSuccess)
                return FA_ERR_CUDA;
        }
    }
    // the call ends when the last copy back has; `stream` is made to wait for it too, so that work the caller
    // queues behind this call is ordered behind the whole of it
    if (cudaEventRecord(h->ev_out_done, h->copy_out) != cudaSuccess || cudaStreamWaitEvent(st, h->ev_out_done, 0) != cudaSuccess)
        return FA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return FA_ERR_CUDA;
    return FA_OK;
}

#ifdef FA_TRACE
// Debug builds only: device buffer of kTraceRoles*kTraceIters*kTraceEvents int64 clock stamps.
fa_status fa_debug_set_trace(fa_handle* h, void* device_buffer) {
    if (!h) return FA_ERR_INVALID_ARG;
    h->trace = static_cast<long long*>(device_buffer);
    return FA_OK;
}
#endif

}  // extern "C"
