// Allocation-free entry point of the library (declared in include/fa.h).
//
// Some callers of this library may not allocate device memory at all: code that runs inside a
// memory plan fixed at start-up (an inference server that hands every byte of HBM to its own
// pools and forbids cudaMalloc afterwards, a real-time loop where an allocation's latency and
// implicit synchronisation are unacceptable, a plug-in that is only given the buffers its host
// application owns).  fa_create allocates (a status word, the split-KV scratch, staging), so
// those callers cannot use the handle-based API.  This entry point needs no handle: the only
// memory the split-KV path needs beyond the caller's Q, K, V, O and lse -- the fp32 partial
// results that the combine kernel merges -- lives in a fixed-size array in the library's own
// device data segment.  The price: the array exists once per GPU that loads the library (it is
// part of the module image, 8 MiB, until the process exits), its size bounds the problems this
// entry point accepts, and all calls share it.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "../../include/fa.h"
#include "fa_common.cuh"
#include "fa_fwd_pipelined.cuh"

namespace {

constexpr size_t kStaticScratchBytes = FA_NOALLOC_SCRATCH_BYTES;

// Partial outputs and partial log-sum-exps of the split-KV kernel.  Device code could name this
// array directly; host code may not pass it to a kernel (on the host the name is a stand-in,
// not a device address) and gets the address with cudaGetSymbolAddress instead.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
// Status of the kernels launched from here ([0] = fa_status, [1] = wait site), written by a device-side wait that runs
// out; the same rule applies: host code asks for its address, kernels get that address.
static __device__ uint32_t g_static_status[2];

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kMaxDevices = 64;

struct DeviceState {          // fixed-size host bookkeeping: no heap
    bool ready = false;
    unsigned char* scratch = nullptr;     // device address of g_static_scratch on this device
    uint32_t* status = nullptr;           // device address of g_static_status on this device
    EncodeTiledFn encode = nullptr;
};
DeviceState g_dev[kMaxDevices];
std::mutex g_dev_mutex;

template <int DQK, int DV>
bool raise_smem_limit() {
    return cudaFuncSetAttribute(fa::fa_fwd_pipelined_kernel<DQK, DV>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize,
                                fa::pipe_smem_bytes<DQK, DV>()) == cudaSuccess;
}

// One-time set-up for the CURRENT device: address of the scratch array on this device, the
// driver's tensor-map encoder, the kernels' shared-memory limit.  No allocating routine is called; with lazy
// module loading the driver places this translation unit's code and data (the 8 MiB array) on the device now.
fa_status setup_current_device(int device) {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    DeviceState& d = g_dev[device];
    if (d.ready) return FA_OK;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) return FA_ERR_CUDA;
    if (major != 10) return FA_ERR_NO_DEVICE;
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
        cudaGetLastError();
        return FA_ERR_CUDA;
    }
    void* sptr = nullptr;
    if (cudaGetSymbolAddress(&sptr, g_static_status) != cudaSuccess || sptr == nullptr) {
        cudaGetLastError();
        return FA_ERR_CUDA;
    }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaGetLastError();
        return FA_ERR_CUDA;
    }
    if (!raise_smem_limit<64, 64>() || !raise_smem_limit<128, 128>() || !raise_smem_limit<192, 128>()) {
        cudaGetLastError();
        return FA_ERR_CUDA;
    }
    d.scratch = static_cast<unsigned char*>(ptr);
    d.status = static_cast<uint32_t*>(sptr);
    d.encode = reinterpret_cast<EncodeTiledFn>(fn);
    d.ready = true;
    return FA_OK;
}

// contiguous [B, H, S, d] bf16 tensor as a 4-D TMA tensor (d, S, H, B)
bool encode_map(EncodeTiledFn encode, CUtensorMap* map, const void* ptr, int d, int S, int H, int B) {
    const cuuint64_t dims[4] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(S),
                                static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(B)};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(d) * 2ull,
                                   static_cast<cuuint64_t>(d) * 2ull * static_cast<cuuint64_t>(S),
                                   static_cast<cuuint64_t>(d) * 2ull * static_cast<cuuint64_t>(S) * static_cast<cuuint64_t>(H)};
    const cuuint32_t box[4] = {static_cast<cuuint32_t>(fa::kChunkCols), static_cast<cuuint32_t>(fa::kTileM), 1u, 1u};
    const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int DQK, int DV>
fa_status launch(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const CUtensorMap& mo,
                 const fa::FwdParams& p,
                 cudaStream_t st) {
    const long long n_ctas = static_cast<long long>((p.n_q_tiles + 1) / 2) * p.Hq * p.B * p.kv_splits;
    if (n_ctas > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;
    fa::fa_fwd_pipelined_kernel<DQK, DV><<<static_cast<unsigned>(n_ctas), fa::PipeCfg<DQK, DV>::kThreads,
                                           fa::pipe_smem_bytes<DQK, DV>(), st>>>(mq, mk, mv, mo, p);
    if (cudaGetLastError() != cudaSuccess) return FA_ERR_CUDA;
    const long long n_rows = static_cast<long long>(p.B) * p.Hq * p.Sq;
    fa::fa_combine_kernel<DV><<<static_cast<unsigned>((n_rows + 3) / 4), 128, 0, st>>>(
        p.o_part, p.lse_part, p.O, p.lse, n_rows, p.kv_splits, p.Hq, p.Sq,
            p.o_stride_b, p.o_stride_h, p.o_stride_s);
    if (cudaGetLastError() != cudaSuccess) return FA_ERR_CUDA;
    return FA_OK;
}

}  // namespace

extern "C" {

size_t fa_noalloc_scratch_bytes(void) { return kStaticScratchBytes; }

fa_status fa_forward_split_noalloc(const void* Q, const void* K, const void* V, void* O, float* lse,
                                   int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv,
                                   int causal, float scale, int kv_splits, void* stream) {
    if (!Q || !K || !V || !O) return FA_ERR_INVALID_ARG;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || dqk <= 0 || dv <= 0) return FA_ERR_INVALID_ARG;
    if (Hq % Hkv != 0 || !isfinite(scale) || scale < 0.f) return FA_ERR_INVALID_ARG;
    if (kv_splits < 2 || kv_splits > 64) return FA_ERR_INVALID_ARG;
    auto misaligned = [](const void* ptr, size_t a) { return (reinterpret_cast<uintptr_t>(ptr) & (a - 1)) != 0; };
    if (misaligned(Q, 16) || misaligned(K, 16) || misaligned(V, 16) || misaligned(O, 16) || (lse && misaligned(lse, 4)))
        return FA_ERR_INVALID_ARG;
    const bool dims_ok = (dqk == 64 && dv == 64) || (dqk == 128 && dv == 128) || (dqk == 192 && dv == 128);
    if (!dims_ok) return FA_ERR_UNSUPPORTED;
    if (static_cast<long long>(B) * Hq > 0x7fffffffLL) return FA_ERR_UNSUPPORTED;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return FA_ERR_NO_DEVICE; }
    if (device < 0 || device >= kMaxDevices) return FA_ERR_UNSUPPORTED;
    fa_status s = setup_current_device(device);     // does its work on the first call per device only
    if (s != FA_OK) return s;
    const DeviceState& dev = g_dev[device];

    if (scale == 0.f) scale = 1.f / sqrtf(static_cast<float>(dqk));
    const int n_q_tiles = (Sq + fa::kTileM - 1) / fa::kTileM;
    int max_tiles = (Sk + fa::kTileN - 1) / fa::kTileN;
    if (causal) {
        const int t = fa::kv_tiles_for_q_tile((n_q_tiles - 1) * fa::kTileM, fa::kTileM, Sq, Sk, 1);
        if (t < max_tiles) max_tiles = t;
    }
    if (max_tiles < 1) max_tiles = 1;
    int splits = kv_splits < max_tiles ? kv_splits : max_tiles;
    if (splits < 2) splits = 2;     // this entry point always takes the split path; an empty split is legal
    const unsigned long long rows = static_cast<unsigned long long>(B) * Hq * Sq;
    const unsigned long long need = static_cast<unsigned long long>(splits) * rows * (dv + 1) * 4ull;
    if (need > kStaticScratchBytes) return FA_ERR_UNSUPPORTED;     // partials exceed the fixed scratch

    CUtensorMap mq, mk, mv, mo;
    if (!encode_map(dev.encode, &mq, Q, dqk, Sq, Hq, B) ||
        !encode_map(dev.encode, &mk, K, dqk, Sk, Hkv, B) ||
        !encode_map(dev.encode, &mv, V, dv, Sk, Hkv, B) ||
        !encode_map(dev.encode, &mo, O, dv, Sq, Hq, B))
        return FA_ERR_CUDA;

    fa::FwdParams p;
    memset(&p, 0, sizeof p);
    p.O = static_cast<__nv_bfloat16*>(O);
    p.o_stride_b = static_cast<long long>(Hq) * Sq * dv;
    p.o_stride_h = static_cast<long long>(Sq) * dv;
    p.o_stride_s = dv;
    p.cu_q = nullptr;
    p.sched_counter = nullptr;
    p.cu_k = nullptr;
    p.total_q = 0;
    p.lse = lse;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.Sq = Sq; p.Sk = Sk;
    p.causal = causal ? 1 : 0;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.n_q_tiles = n_q_tiles;
    p.heads_per_group = B * Hq;                 // short problems: everything fits in L2
    p.status = dev.status;                      // a wait that runs out leaves its code here (fa_noalloc_last_status)
    p.wait_limit_ns = 2000ull * 1000000ull;
    p.kv_splits = splits;
    p.tiles_per_split = (max_tiles + splits - 1) / splits;
    // Every (split, row) slot below is overwritten by exactly one CTA of this call, so nothing in
    // the array has to be cleared first, whatever an earlier call left there.
    p.o_part = reinterpret_cast<float*>(dev.scratch);
    p.lse_part = p.o_part + static_cast<size_t>(splits) * rows * dv;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dqk == 64) return launch<64, 64>(mq, mk, mv, mo, p, st);
    if (dqk == 128) return launch<128, 128>(mq, mk, mv, mo, p, st);
    return launch<192, 128>(mq, mk, mv, mo, p, st);
}

fa_status fa_noalloc_last_status(uint32_t* detail) {
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return FA_ERR_NO_DEVICE; }
    if (device < 0 || device >= kMaxDevices) return FA_ERR_UNSUPPORTED;
    if (detail) *detail = 0;
    if (!g_dev[device].ready) return FA_OK;      // nothing has been launched from here on this device
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return FA_ERR_CUDA; }
    uint32_t words[2] = {0, 0};
    if (cudaMemcpyFromSymbol(words, g_static_status, sizeof words) != cudaSuccess) { cudaGetLastError(); return FA_ERR_CUDA; }
    if (words[0] != 0) {
        const uint32_t zero[2] = {0, 0};
        if (cudaMemcpyToSymbol(g_static_status, zero, sizeof zero) != cudaSuccess) { cudaGetLastError(); return FA_ERR_CUDA; }
    }
    if (detail) *detail = words[1];
    return static_cast<fa_status>(words[0]);
}

}  // extern "C"
