/*
 * fa.h -- C ABI of the B200 (sm_100a) fused attention forward library.
 *
 * The library computes, for every batch b, query head hq and query row i,
 *
 *     O[b,hq,i,:] = softmax_j( scale * <Q[b,hq,i,:], K[b,kvh,j,:]> ) . V[b,kvh,:,:]
 *     lse[b,hq,i] = ln sum_j exp( scale * <Q[b,hq,i,:], K[b,kvh,j,:]> )
 *
 * which is Eq. 1 of the paper (scaled dot-product attention, Section 2.1)
 * replicated over heads, evaluated by the fused online-softmax recurrence of
 * Algorithm 1 (running row maximum u, running row sum s, unnormalised
 * accumulator G', one division at the end), so that the Sq x Sk score matrix
 * never leaves the SM.  `causal` selects the mask step of Algorithm 1: key j is
 * visible to query i iff j <= i + (Sk - Sq) (for Sq == Sk: a token sees itself
 * and its predecessors).  Grouped-query attention (Section 4.4): query head hq
 * reads kv head kvh = hq / (Hq / Hkv).  Data are bfloat16 as in the paper's
 * evaluation (Section 5.1); scores, the softmax state and both accumulators
 * are fp32.  lse is not a paper output: it carries the (u, s) pair that
 * Algorithm 1 returns, as u + ln s, in natural-log units of the scaled scores.
 *
 * Layouts (row-major, contiguous, no padding):
 *     Q   [B, Hq,  Sq, dqk]  bf16        K [B, Hkv, Sk, dqk] bf16
 *     V   [B, Hkv, Sk, dv ]  bf16        O [B, Hq,  Sq, dv ] bf16
 *     lse [B, Hq,  Sq]       fp32
 * Rows with no visible key (possible only when causal and Sq > Sk) get
 * O = 0 and lse = -inf.
 *
 * Supported head sizes: (dqk, dv) in {(64,64), (128,128), (192,128)}.
 *
 * Threading: a handle must not be used from two host threads at once.
 * All functions return a status code; nothing throws, aborts or prints.
 */
#ifndef FA_B200_H_
#define FA_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fa_handle fa_handle; /* opaque; created by fa_create, freed by fa_destroy */

typedef enum fa_status {
    FA_OK = 0,
    FA_ERR_INVALID_ARG = 1,    /* NULL/misaligned pointer, non-positive size, Hq % Hkv != 0, bad scale */
    FA_ERR_UNSUPPORTED = 2,    /* head sizes or extents the kernels do not cover                     */
    FA_ERR_CUDA = 3,           /* a CUDA runtime/driver call failed (launch, copy, allocation)       */
    FA_ERR_DEVICE_TIMEOUT = 4, /* a bounded device-side wait ran out; the results are invalid        */
    FA_ERR_NO_DEVICE = 5,      /* no CUDA device, or the device is not compute capability 10.x       */
    FA_ERR_OOM = 6             /* host or device allocation failed                                   */
} fa_status;

/* fa_config.flags: run the serialised cross-check kernel (one tile in flight, no overlap
 * between loads, MMAs and softmax) instead of the pipelined one.  Same results up to
 * rounding order; much slower.  Meant for tests. */
#define FA_FLAG_SERIAL_KERNEL 1u
/* fa_config.flags, test hook for the failure path: the loading thread of whichever kernel runs
 * (every attention kernel of the library honours it, the 8-bit ones included) leaves out the load
 * of its CTA's first V tile, so the wait for it runs into the device-side limit
 * (fa_config.wait_limit_ms).  The kernel then returns normally, results are invalid and
 * fa_last_status reports FA_ERR_DEVICE_TIMEOUT; the context and the handle stay usable.  Nothing
 * faults, traps or spins without bound.  Use with a short wait_limit_ms on a tiny problem.
 * fa_debug_set_drop_v_load switches the hook on and off for an existing handle. */
#define FA_FLAG_DEBUG_DROP_V_LOAD 2u
/* fa_config.flags: launch the kernels the ordinary way.  By default the pipelined kernel (and the
 * split-KV combine kernel) are launched with programmatic stream serialisation: the GPU may
 * schedule their CTAs while the kernel before them in the stream is still draining, and they
 * wait on the device for that kernel's completion before they read or write global memory.
 * Results and ordering guarantees are the same either way; the default saves the stream's
 * completion-to-launch latency (a few microseconds per launch). */
#define FA_FLAG_NO_DEPENDENT_LAUNCH 4u
/* fa_config.flags: kernel choice.  The library runs problems with many short work items (at
 * least three pairs of query tiles per SM, at most 64 K/V tiles each, 16 at head size 64;
 * packed batches counted by their longest sequence) on a persistent variant of the pipelined
 * kernel (one CTA per SM walking a list of items) and everything else on the one-item-per-CTA kernel.  These two flags override the choice where
 * both kernels apply (head sizes 64 and 128, no split-KV); results are bit-identical.  The stream kernel
 * (FA_FLAG_STREAM_KERNEL below) has a persistent form of its own for fixed-length launches with at least three
 * one-tile items per SM of at most 32 K/V tiles each (csrc/fa_fwd_stream_persistent.cuh; any number and length of
 * items with FA_FLAG_FORCE_PERSISTENT), under the same two flags and with the same guarantee. */
#define FA_FLAG_NO_PERSISTENT 8u
#define FA_FLAG_FORCE_PERSISTENT 16u
/* A third tiling: one query tile per CTA with its K/V tiles streamed through both softmax
 * warpgroups (csrc/fa_fwd_stream.cuh).  It doubles the number of CTAs and shortens each one's
 * dependency chain, which wins when the pair tiling leaves SMs idle or its longest CTA dominates
 * (under about one wave of pairs: short sequences, few heads); the library estimates both and
 * picks it with a 10 % margin (each with its own split-KV count); at head sizes 192/128,
 * where the pair kernel is short of shared memory, it is ahead at every size.  These flags force
 * it on (fixed-length problems) or off. */
#define FA_FLAG_STREAM_KERNEL 32u
#define FA_FLAG_NO_STREAM_KERNEL 64u
/* With at most 64 queries per sequence and several query heads per K/V head (decoding with
 * grouped-query attention), the stream kernel puts the rows of several heads of a group into one
 * query tile, so every K/V tile is fetched and multiplied once for all of them: the largest
 * divisor h of the group size with h * Sq <= 128 heads share a tile.  Results are those of the
 * unpacked launch up to fp32 rounding order (a row's arithmetic does not depend on its
 * neighbours).  This flag turns the packing off.  It also turns off the pairing of heads on the
 * tilings with two query tiles per CTA (an even group size under a causal mask or with an odd
 * number of query tiles: the CTA's tiles are the same query tile of two adjacent heads of a
 * group instead of two adjacent query tiles of one head; results bit-identical either way). */
#define FA_FLAG_NO_HEAD_PACKING 128u
/* fa_config.flags: at head size 128 the tilings with two query tiles per CTA have two generations of
 * kernels: csrc/fa_fwd_pair.cuh and its persistent form csrc/fa_fwd_pair_persistent.cuh (the default:
 * one MMA-issuing thread that probes its barriers from inside the blocks of MMAs, no correction
 * warpgroup) and the older csrc/fa_fwd_pipelined.cuh and csrc/fa_fwd_persistent.cuh, which this flag
 * selects.  Same results, bit for bit.  Meant for tests and A/B timing. */
#define FA_FLAG_LEGACY_PAIR_KERNEL 256u
/* fa_config.flags: run fixed-length problems without split-KV at head sizes 128 and 192/128 on the
 * kernel that pairs two SMs (a cluster of two CTAs with one query tile each, every MMA issued once
 * for both as a two-CTA tcgen05.mma, each CTA holding half of every K/V tile).  Its two softmax
 * warpgroups keep separate partial results for the even and the odd K/V tiles and merge them at
 * the end, so its output agrees with the other kernels' to rounding, not bit for bit. */
#define FA_FLAG_TWO_CTA_KERNEL 512u
/* fa_config.flags: run the same class of problems on the kernel that gives a pair of SMs FOUR query tiles (two
 * per CTA, as in the pair kernels, every MMA a two-CTA tcgen05.mma over one tile of each CTA): csrc/fa_fwd_quad.cuh.
 * Takes precedence over FA_FLAG_TWO_CTA_KERNEL. */
#define FA_FLAG_QUAD_KERNEL 1024u

/* Optional creation parameters.  Zero-initialise, set struct_size = sizeof(fa_config). */
typedef struct fa_config {
    uint32_t struct_size;     /* sizeof(fa_config) of the caller's header                      */
    int32_t device;           /* CUDA device ordinal; -1 = the calling thread's current device */
    uint32_t flags;           /* bitwise OR of FA_FLAG_*; other bits must be 0                 */
    uint32_t wait_limit_ms;   /* limit of every device-side wait; 0 = default (2000 ms)        */
    uint32_t kv_splits;       /* split-KV: 0 = library decides, 1 = never split, 2..256 = use n
                                 splits whenever the scratch buffer can hold the partials      */
    uint64_t scratch_bytes;   /* device scratch for split-KV partials, allocated by fa_create;
                                 0 = default (32 MiB)                                          */
} fa_config;

/*
 * Split-KV (the spatial decomposition of Algorithm 2: the key/value range of a query tile is
 * partitioned over C CTAs, each running Algorithm 1 on its part, and the partial results are
 * merged with the online-softmax reduction): used when a problem has too few query tiles to
 * fill the GPU (short Sq with long Sk).  The partials (fp32 O_c and lse_c per query row) live
 * in the handle's scratch buffer, and a second small kernel merges them.  The printed merge of
 * Algorithm 2 rescales with the previous partial's maximum; the library uses the corrected
 * form lse = ln sum_c exp(lse_c), O = sum_c exp(lse_c - lse) O_c.
 */

/*
 * Create a handle bound to one device.  `cfg` may be NULL (defaults, current
 * device).  The handle owns a small status word (pinned host memory mapped to
 * the device), a cache of TMA tensor maps keyed by (pointer, shape), the split-KV
 * scratch buffer and the staging buffers of fa_forward_host.  Allocates; call
 * outside stream capture.  A struct_size smaller than the current fa_config is accepted:
 * missing trailing fields take their defaults.
 */
fa_status fa_create(fa_handle** out, const fa_config* cfg);

/*
 * Fused attention forward (Eq. 1 evaluated by Algorithm 1; causal mask,
 * GQA head sharing and lse as described at the top of this file).
 *
 *   Q, K, V  device pointers to bf16, 16-byte aligned, layouts as above; read only.
 *   O        device pointer to bf16, 16-byte aligned; every element is overwritten.
 *   lse      device pointer to fp32, 4-byte aligned, or NULL to skip it.
 *   B, Hq, Hkv, Sq, Sk, dqk, dv   extents; all > 0; Hq % Hkv == 0.  Sq and Sk need
 *            not be multiples of the 128-row tile.
 *   causal   0 = every key visible; non-zero = key j visible iff j <= i + (Sk - Sq).
 *   scale    multiplier of the dot products; 0.0f selects 1/sqrt(dqk) (Eq. 1).
 *            Must be finite and >= 0.
 *   stream   a cudaStream_t (NULL = the legacy default stream) of the handle's device.
 *
 * The call is asynchronous: it validates, enqueues the kernel on `stream` and
 * returns.  The caller owns all buffers and keeps them alive until the stream
 * has passed the kernel; O must not alias an input.  The library does not
 * synchronise and does not allocate device memory here (split-KV partials use the
 * scratch buffer allocated by fa_create; launches through one handle must therefore not
 * overlap on the device: use one handle per stream).  Argument and launch
 * errors are returned at once; a device-side timeout shows up in
 * fa_last_status after the caller has synchronised the stream.
 */
fa_status fa_forward(fa_handle* h,
                     const void* Q, const void* K, const void* V,
                     void* O, float* lse,
                     int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv,
                     int causal, float scale, void* stream);

/*
 * fa_forward for tensors that are not contiguous [B, H, S, d] (Eq. 1 fixes no memory layout; a
 * projection kernel usually leaves Q, K, V as [B, S, H, d]).  Each strides argument points to three
 * int64 values {batch stride, head stride, row stride} in ELEMENTS; element (b, h, s, c) of a
 * tensor sits at base + b*batch + h*head + s*row + c, the last dimension is contiguous.  Every
 * stride must be positive and a multiple of 8 elements (16 bytes: the TMA unit and the 16-byte
 * output stores require it), and a row stride must not be smaller than the head size.  lse stays
 * contiguous [B, Hq, Sq].  Everything else is as for fa_forward; FA_ERR_INVALID_ARG if the strides
 * cannot be expressed.
 */
fa_status fa_forward_strided(fa_handle* h,
                             const void* Q, const void* K, const void* V,
                             void* O, float* lse,
                             int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv,
                             int causal, float scale,
                             const int64_t* q_strides, const int64_t* k_strides,
                             const int64_t* v_strides, const int64_t* o_strides,
                             void* stream);

/*
 * Eq. 1 on a batch of sequences of different lengths, packed without padding (the paper's
 * sequence-length sweeps run one length at a time; serving batches mix them).  Sequence b owns
 * rows [cu_seqlens_q[b], cu_seqlens_q[b+1]) of Q and O and rows [cu_seqlens_k[b],
 * cu_seqlens_k[b+1]) of K and V.
 *   Q [total_q, Hq, dqk], K [total_k, Hkv, dqk], V [total_k, Hkv, dv], O [total_q, Hq, dv]: bf16,
 *     contiguous, DEVICE pointers, 16-byte aligned.
 *   lse [Hq, total_q] fp32 DEVICE pointer or NULL.
 *   cu_seqlens_q, cu_seqlens_k: DEVICE arrays of B+1 int32, non-decreasing, starting at 0 and
 *     ending at total_q / total_k.  The host never reads them (no synchronisation); the caller
 *     vouches for their contents.
 *   max_sq: an upper bound of the query lengths (sizes the grid).  Rows of a sequence past max_sq
 *     are not computed and their O and lse are left untouched.
 * The causal mask is aligned to the end of each sequence: key j of sequence b is visible to its
 * query i iff j <= i + (Sk_b - Sq_b).  A sequence with no keys, and any row with no visible key,
 * gets O = 0 and lse = -inf; a sequence with no queries writes nothing.  Rows of K/V past the end
 * of a sequence take no part in the result, but must hold finite numbers where they belong to the
 * next sequence (they are multiplied by a zero probability).  The K/V range is split over CTAs
 * only for batches with a single 128-row query tile per sequence (max_sq <= 128) that would
 * leave most SMs idle; every CTA then cuts its own sequence into the equal shares.  With max_sq <= 64 and several query heads per K/V head the heads of a group
 * share a query tile (see FA_FLAG_NO_HEAD_PACKING): a decode step over sequences of different
 * lengths then reads every K/V head once.  Errors as for fa_forward.
 */
fa_status fa_forward_varlen(fa_handle* h,
                            const void* Q, const void* K, const void* V,
                            void* O, float* lse,
                            const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k,
                            int B, int total_q, int total_k, int max_sq,
                            int Hq, int Hkv, int dqk, int dv,
                            int causal, float scale, void* stream);

/*
 * Block-scaled 8-bit variant (the counterpart of the paper's block floating-point data path,
 * Section 3): Q8, K8, V8 hold e4m3 values (one byte each, the "fn" encoding without infinities),
 * contiguous [B, H, S, d] DEVICE tensors with d = 64 or 128, 16-byte aligned.  The represented tensors are
 *   Q[b,h,i,:] = q_scale[b,h,i/128] * Q8[b,h,i,:]     q_scale [B, Hq,  ceil(Sq/128)]
 *   K[b,h,j,:] = k_scale[b,h,j/128] * K8[b,h,j,:]     k_scale [B, Hkv, ceil(Sk/128)]
 *   V[b,h,j,:] = v_scale[b,h]       * V8[b,h,j,:]     v_scale [B, Hkv]
 * with positive fp32 scales in DEVICE memory (a NULL scale pointer means 1).  Both contractions
 * run on the 8-bit tensor-core path with fp32 accumulation; the probabilities are rounded to e4m3
 * before the second one (the row sums use the unrounded values).  O is bf16 [B, Hq, Sq, d], lse
 * fp32 [B, Hq, Sq] or NULL, both of Eq. 1 applied to the represented Q, K, V.  Head sizes 64 and
 * 128, and d = 192 for the 192/128 shapes (Q8 and K8 with 192 columns, V8 and O with 128; stream
 * tiling with one head per query tile); other sizes, and handles created with FA_FLAG_SERIAL_KERNEL,
 * return FA_ERR_UNSUPPORTED.  The
 * tiling is planned as for fa_forward (pair or stream tiling, split-KV and shared query tiles for
 * grouped heads on the stream tiling; the partials use the handle's scratch buffer); with shared
 * query tiles of at most 64 rows the rows are additionally processed as two or four copies that
 * each take a slice of every K/V tile's keys and are merged like split-KV partials.  Other
 * arguments and errors as for fa_forward.
 */
fa_status fa_forward_fp8(fa_handle* h,
                         const void* Q8, const void* K8, const void* V8,
                         const float* q_scale, const float* k_scale, const float* v_scale,
                         void* O, float* lse,
                         int B, int Hq, int Hkv, int Sq, int Sk, int d,
                         int causal, float scale, void* stream);

/*
 * MX form of the 8-bit variant (microscaling: the closest counterpart on this GPU of a block
 * floating-point format, Section 3 / Table 1 of the paper): e4m3 values with one e8m0 scale
 * 2^(byte - 127) per 32 elements ALONG EACH CONTRACTION, applied inside the tensor-core instruction
 * (tcgen05.mma kind::mxf8f6f4 with block scaling).  Q8, K8, V8 as for fa_forward_fp8.  The
 * represented tensors are
 *   Q[b,h,i,c] = 2^(eq - 127) * Q8[b,h,i,c]   eq = scale of (row i, columns 32*(c/32) .. +31)
 *   K[b,h,j,c] = 2^(ek - 127) * K8[b,h,j,c]   ek = scale of (key j, columns 32*(c/32) .. +31)
 *   V[b,h,j,c] = 2^(ev - 127) * V8[b,h,j,c]   ev = scale of (column c, keys 32*(j/32) .. +31)
 * and the scales are passed in the layout the tensor core reads them in, one 512-byte atom per
 * 128-row tile (DEVICE memory, 16-byte aligned, uint8):
 *   q_sf [B, Hq,  ceil(Sq/128), 512]   byte (r%32)*16 + (r/32)*4 + kb : row 128*t + r, column block kb
 *   k_sf [B, Hkv, ceil(Sk/128), 512]   byte (r%32)*16 + (r/32)*4 + kb : key 128*t + r, column block kb
 *   v_sf [B, Hkv, ceil(Sk/128), 512]   byte (c%32)*16 + (c/32)*4 + kb : column c, keys 128*t + 32*kb .. +31
 * (d = 64 uses kb = 0, 1 of Q and K and c < 64 of V; unused bytes, and those of rows past the end
 * of a tensor, must still be valid scales, e.g. 127: 255 is NaN.)  The probabilities are rounded to
 * e4m3 with scale 1 before the second contraction, as in fa_forward_fp8.  Runs on the stream tiling
 * (one head per query tile, split-KV where the plan wants it).  O, lse, other arguments and errors
 * as for fa_forward_fp8.
 */
fa_status fa_forward_mxfp8(fa_handle* h,
                           const void* Q8, const void* K8, const void* V8,
                           const uint8_t* q_sf, const uint8_t* k_sf, const uint8_t* v_sf,
                           void* O, float* lse,
                           int B, int Hq, int Hkv, int Sq, int Sk, int d,
                           int causal, float scale, void* stream);

/*
 * What the library would launch for a problem: which kernel (tiling), how many K/V splits, how
 * many CTAs, and the two run-time estimates behind the choice (0 when none was needed).  A pure
 * host function: no handle, no device, no CUDA call; `num_sms` is the SM count to plan for (148 on
 * B200) and `cfg` the creation parameters a handle would have (NULL = defaults; its device field is
 * ignored).  `varlen` != 0 plans fa_forward_varlen with Sq = max_sq and Sk = the mean key length.
 * The tile schedule is the first step of the path (one CTA per pair of query tiles in the paper's
 * mapping, Section 4); here it is chosen per launch, and this call makes the choice inspectable.
 * Returns FA_ERR_UNSUPPORTED for head sizes the kernels do not have, FA_ERR_INVALID_ARG otherwise.
 */
typedef struct fa_plan_info {
    const char* kernel;          /* "fa_fwd_pipelined", "fa_fwd_stream", "fa_fwd_persistent", "fa_fwd_simple" */
    int32_t kv_splits;           /* CTAs per work item along the K/V range (1 = no split)        */
    int64_t ctas;                /* grid size of the attention kernel                            */
    int32_t heads_per_tile;      /* query heads sharing a query tile (1 = none; see FA_FLAG_NO_HEAD_PACKING) */
    double estimate_pair_us;     /* estimated time with one CTA per pair of query tiles          */
    double estimate_stream_us;   /* estimated time with one CTA per query tile                   */
} fa_plan_info;
fa_status fa_plan(int num_sms, const fa_config* cfg, int varlen,
                  int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv, int causal,
                  fa_plan_info* out);

/*
 * The same operation with HOST buffers (same layouts and types): copies Q, K, V
 * to staging memory owned by the handle, runs fa_forward, copies O (and lse if
 * not NULL) back, and synchronises `stream` before returning.  Problems of 256 MiB
 * and more (all five tensors) are cut into up to 16 chunks of whole (batch, K/V head)
 * units, which are independent and contiguous in every tensor: the copies of the
 * next chunk in and of the previous chunk out run on two copy streams of the handle
 * under the kernel of the current chunk, which runs on `stream`; work queued on
 * `stream` before the call precedes all of it, work queued after it follows all of
 * it.  Smaller problems go through `stream` in one piece.  Pinned host buffers give
 * the full copy bandwidth and the overlap; pageable ones work.  The staging buffers
 * grow on demand (device allocation on the first call and whenever a larger problem
 * arrives; the copy streams and events are created by the first large call) and are
 * freed by fa_destroy.
 */
fa_status fa_forward_host(fa_handle* h,
                          const void* Q_host, const void* K_host, const void* V_host,
                          void* O_host, float* lse_host,
                          int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv,
                          int causal, float scale, void* stream);

/*
 * Device-side status of the kernels launched through `h` so far: FA_OK, or
 * FA_ERR_DEVICE_TIMEOUT if any bounded wait (mbarrier, TMEM allocation) ran
 * out since the handle was created or the status was last read (reading
 * clears it).  Synchronises nothing: meaningful after the caller has
 * synchronised the stream(s) it launched on.  `detail`, if not NULL, receives
 * a diagnostic word (role and barrier that gave up; 0 when FA_OK).
 */
fa_status fa_last_status(fa_handle* h, uint32_t* detail);

/* Test hook: switches FA_FLAG_DEBUG_DROP_V_LOAD on (enabled != 0) or off for launches made through `h` from now on,
 * so that a test can make one launch run into its wait limit and check that the next one through the same handle
 * is correct.  When fa_last_status reports an error it also puts the persistent kernel's work-item counter, which a
 * launch that gave up leaves half-way, back to zero: call it (after synchronising) before launching again. */
fa_status fa_debug_set_drop_v_load(fa_handle* h, int enabled);

/* Free everything the handle owns.  fa_destroy(NULL) returns FA_OK. */
fa_status fa_destroy(fa_handle* h);

/* Static, NUL-terminated description of a status code. */
const char* fa_strerror(fa_status s);

/*
 * Introspection used by tests and the benchmark: number of kernel launches
 * issued through the handle so far (a split-KV forward is two launches), the
 * name of the kernel variant the last fa_forward selected (static string; ""
 * before the first call), and the number of K/V splits it used.
 */
uint64_t fa_launch_count(const fa_handle* h);
const char* fa_last_kernel_name(const fa_handle* h);
int fa_last_kv_splits(const fa_handle* h);   /* K/V splits the last fa_forward used (1 = none) */

/*
 * Allocation-free split-KV forward.  (The paper has no counterpart: this entry point exists for
 * callers that cannot allocate, it is not a step of the paper's method.)
 *
 * Who needs it: code that must not call cudaMalloc or any allocating routine once it is running --
 * a server that has handed all of HBM to its own pools, a real-time loop that cannot afford an
 * allocation's latency and implicit synchronisation, a plug-in that only gets its host's buffers.
 * fa_create allocates, so such callers cannot hold a handle; this function takes none.
 *
 * It computes exactly what fa_forward computes with kv_splits-way split-KV.  The fp32 partials that
 * the combine kernel merges live in an array of FA_NOALLOC_SCRATCH_BYTES (8 MiB) in the library's
 * device data segment: every GPU that loads the library carries that array until the process
 * exits.  Consequences:
 *   - the partials must fit: splits * B*Hq*Sq * (dv + 1) * 4 bytes <= FA_NOALLOC_SCRATCH_BYTES, where
 *     splits = min(kv_splits, number of K/V tiles) (at least 2); larger problems are rejected with
 *     FA_ERR_UNSUPPORTED and nothing is launched;
 *   - all calls share the array and it keeps the previous call's contents.  Nothing needs clearing
 *     (each call overwrites every slot it later reads), but two calls that overlap on the device --
 *     different streams, or different host threads -- race on it: serialise them;
 *   - the first call on a device performs a one-time set-up for that device (looks up the array's
 *     device address, the driver's tensor-map encoder, raises the kernels' shared-memory limit).
 *     Make that first call with the device current and before any stream capture begins.  With CUDA's
 *     lazy module loading that first call is also when the driver places this part of the library on
 *     the device, code and the 8 MiB array included: a caller that hands all of the device's memory to
 *     its own pools should make one small call BEFORE it freezes its memory plan.  Later calls do not
 *     allocate.
 * The library itself calls no allocating routine here (no cudaMalloc, no host heap).  Arguments as for
 * fa_forward; kv_splits in [2, 64]; device pointers; the work is enqueued on `stream` of the CURRENT
 * device and the call returns without synchronising.  A device-side wait that runs out is recorded in a
 * status word that also lives in the library's device data; fa_noalloc_last_status reads it.
 */
#define FA_NOALLOC_SCRATCH_BYTES (8u << 20)
fa_status fa_forward_split_noalloc(const void* Q, const void* K, const void* V,
                                   void* O, float* lse,
                                   int B, int Hq, int Hkv, int Sq, int Sk, int dqk, int dv,
                                   int causal, float scale, int kv_splits, void* stream);
size_t fa_noalloc_scratch_bytes(void);   /* FA_NOALLOC_SCRATCH_BYTES as built into the library */
/* (no paper counterpart) Status of the fa_forward_split_noalloc calls on the CURRENT device since the last call of this
 * function: synchronises the device, returns FA_OK or FA_ERR_DEVICE_TIMEOUT (with the wait site in *detail when
 * detail is not NULL) and clears the word.  Allocates nothing.  The word is shared by all calls, like the array. */
fa_status fa_noalloc_last_status(uint32_t* detail);

#ifdef __cplusplus
}
#endif
#endif /* FA_B200_H_ */
