// Internal declarations shared by the translation units of libpatchkv (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <mutex>
#include <string>
#include <utility>
#include <vector>

#include "patchkv.h"

namespace patchkv {

enum { FMT_BF16 = 0, FMT_INT8 = 1, FMT_INT4 = 2 };

__host__ __device__ inline int k_format(int tag) {
    return tag == PATCHKV_TAG_BF16 ? FMT_BF16 : (tag == PATCHKV_TAG_K4V4 ? FMT_INT4 : FMT_INT8);
}
__host__ __device__ inline int v_format(int tag) {
    return tag == PATCHKV_TAG_BF16 ? FMT_BF16 : (tag == PATCHKV_TAG_INT8 ? FMT_INT8 : FMT_INT4);
}
// Code bytes and scale bytes of one K or V section holding `elems` elements.
__host__ __device__ inline uint64_t code_bytes(int fmt, uint64_t elems) {
    return fmt == FMT_BF16 ? 2 * elems : (fmt == FMT_INT8 ? elems : elems / 2);
}
__host__ __device__ inline uint64_t scale_bytes(int fmt, uint64_t elems, int group) {
    return fmt == FMT_BF16 ? 0 : 2 * (elems / (uint64_t)group);
}
__host__ __device__ inline uint64_t record_bytes(int tag, uint64_t elems, int group) {
    if (tag < 0 || tag > PATCHKV_TAG_K4V4) return 0;
    const int kf = k_format(tag), vf = v_format(tag);
    return code_bytes(kf, elems) + scale_bytes(kf, elems, group) + code_bytes(vf, elems) + scale_bytes(vf, elems, group);
}

// Two fp32 lanes per instruction (sm_100 packed fp32): same IEEE result per lane as the scalar operation,
// each lane rounded on its own, no fusion.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
// ---- shared-memory barriers, bulk asynchronous copies and shared loads (sm_90+ PTX) -------------------------------
constexpr uint32_t kWaitLimit = 1u << 22;      // polls before a barrier wait gives up

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the limit ran out (the abort flag is then raised) or another role aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t limit = kWaitLimit) {
    for (uint32_t i = 0; i < limit; i++) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (i > 32) __nanosleep(40);
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint16_t lds16(uint32_t a) {
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
    return v;
}

// Programmatic dependent launch (sm_90+).  A kernel launched with launch_pdl may be brought onto the SMs while the kernel
// in front of it in the stream is still running; it calls pdl_wait() before it touches global memory, which returns
// once that kernel has completed and its writes are visible.  pdl_trigger() tells the runtime that the kernel behind
// this one may be brought on.  Both are no-ops for kernels launched the ordinary way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Exclusive prefix sum of v over a CTA of kScanThreads threads; *total receives the CTA sum.  `warp_sums` is 33 ints
// of shared memory.  Every thread of the CTA has to call it (it contains CTA-wide barriers).
constexpr int kScanThreads = 1024;
__device__ __forceinline__ int cta_exclusive_scan(int v, int* warp_sums, int* total) {
    const unsigned lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= (unsigned)d) inc += o;
    }
    __syncthreads();                                 // warp_sums free to overwrite
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const int w = warp_sums[lane];               // kScanThreads / 32 = 32 warps: one per lane
        int winc = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xFFFFFFFFu, winc, d);
            if (lane >= (unsigned)d) winc += o;
        }
        warp_sums[lane] = winc - w;                  // exclusive offset of each warp
        if (lane == 31) warp_sums[32] = winc;
    }
    __syncthreads();
    *total = warp_sums[32];
    return warp_sums[warp] + inc - v;
}

// One session as the restore kernel sees it (all pointers device memory).
struct SessionDev {
    const int32_t* block_table;
    const uint8_t* tags;
    const unsigned long long* blk_off;
    const void* const* layer_payload;
    const unsigned long long* layer_bytes;
    const int32_t* reuse_idx;
    const int32_t* reuse_cnt;
    int32_t n, nb, delta, dst_shift, n_table;
    int32_t list_nb;        // row stride of reuse_idx, and work items per layer (nb unless the host path split the list)
    int32_t item_begin;     // first work item of this session in the launch's item numbering
};

struct RestoreParams {
    // geometry
    int32_t L, H, D, Dr, rope_style, B, P, G;
    int32_t scalar_only;    // 1: a geometry only the element-wise kernel takes
    // pool
    uint16_t* k_base;
    uint16_t* v_base;
    long long stride_layer, stride_page, stride_token, stride_head;
    int32_t n_pages;
    // work: items are (session, layer in [layer_begin, layer_end), position r in the reuse list)
    int32_t n_sessions, layer_begin, layer_end, total_items;
    int32_t grid_cap;       // > 0: launch at most this many CTAs (the host path's side launch that reads over the link)
    int32_t* status;        // device status word
    int32_t* sched;         // this launch's slot of work counters: [0] blocks handed out, [1] CTAs that have left
                            // (the last CTA to leave zeroes both, so the slot starts the next launch at zero)
    uint32_t wait_limit;    // polls before a barrier wait gives up (kWaitLimit unless a self-test shortened it)
    int32_t stall_after;    // self-test only: consumer group 0 of every CTA withholds the `empty` arrival of its
                            // unit number stall_after (-1: never)
    // bulk-copy pipeline: bytes of a stage and of its data area, ring depth, tokens per unit of a section slice, and
    // per tag how many whole records one unit may carry (0: the record is staged a section slice at a time)
    int32_t unit_tokens, stage_data_bytes, stage_bytes, n_stages;
    int32_t unit_records[4];
    int32_t B_shift, P_shift;       // log2 of B / P when a power of two, else -1
    int32_t round_cap, round_div;   // a round of self-scheduled blocks: min(round_cap, left / (round_div * CTAs)), at least 1
    uint32_t blk_codes[3], blk_scales[3], tok_codes[3], tok_scales[3];   // bytes per block / per token, by format
    uint32_t rec_bytes[4];  // bytes of a block record, by tag
    SessionDev s[PATCHKV_MAX_SESSIONS];
    // cos / sin of delta * theta_i per session, fp32, built on the host in double
    float cs[PATCHKV_MAX_SESSIONS][2][PATCHKV_MAX_ROTARY_DIM / 2];
};

struct Staging {
    void* base = nullptr;
    size_t bytes = 0;
    cudaEvent_t copied = nullptr;   // recorded on the copy stream when the slot's copies are enqueued
    cudaEvent_t freed = nullptr;    // recorded on the decode stream after the kernel that read the slot
};

}  // namespace patchkv

struct patchkv_ctx {
    int device = 0;
    int sm_count = 0;
    int staging_slots = 4;
    int flags = 0;
    int max_smem_optin = 0;
    int smem_per_sm = 0;
    uint64_t merge_gap = 64 * 1024;
    int direct_percent = 48;                // hybrid host path: share of a layer's bytes that its side launch reads directly ...
    uint64_t pause_fill_bytes = 100 * 1024; // ... plus this much per copy left to the engine (half of what the side launch
                                            // reads during the engine's pause between two copies, ~4 us at ~50 GB/s)
    int direct_ctas = 4;                    // hybrid host path: CTAs of a side launch
    cudaStream_t copy_stream = nullptr, decode_stream = nullptr, direct_stream = nullptr;
    cudaEvent_t ev_begin = nullptr, ev_done = nullptr, ev_direct = nullptr;
    int32_t* d_status = nullptr;
    // Work-counter slots of the restore pipeline (two words each, zero between launches: the kernel resets its
    // own slot).  A slot is private to whatever serialises the launches that use it: slot 0 belongs to the internal
    // decode stream, every caller stream gets a slot of its own on first use, and a launch recorded into a CUDA
    // graph gets a slot that nothing else ever uses.
    int32_t* d_sched = nullptr;
    std::vector<std::pair<uint64_t, uint64_t>> sched_streams;   // (stream handle, host thread for per-thread streams)
    int sched_captured = 0;         // slots handed to captured launches so far
    // self-test: the next pipeline launch runs with this wait limit and stalls one consumer group (see patchkv.h)
    uint32_t selftest_wait_limit = 0;
    int32_t selftest_stall_after = -1;
    // select workspace (block masses when the caller gives no mass_out; summed mass for LAYERS_SHARED)
    unsigned long long* d_mass_ws = nullptr;
    size_t mass_ws_elems = 0;
    // restore_from_host: staging ring, metadata arenas
    std::vector<patchkv::Staging> slots;
    uint8_t* d_meta = nullptr;
    uint8_t* h_meta = nullptr;      // pinned mirror
    uint8_t* h_meta_alias = nullptr;    // its device alias (the host path's kernels read their reuse lists there)
    size_t meta_bytes = 0;
    bool host_call_pending = false;
    std::string last_error;
    std::mutex mu;
};

namespace patchkv {

constexpr int kSchedStreamSlots = 192;      // slots 0, 1: the internal decode and direct streams; 2 .. 191: caller streams
constexpr int kSchedCaptureSlots = 320;     // launches recorded into CUDA graphs over the life of a context
constexpr int kSchedSlots = kSchedStreamSlots + kSchedCaptureSlots;

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

inline int fail(patchkv_ctx* ctx, int code, const std::string& msg) {
    if (ctx) ctx->last_error = msg;
    return code;
}

#define PKV_CUDA(ctx, expr)                                                                       \
    do {                                                                                          \
        cudaError_t e_ = (expr);                                                                  \
        if (e_ != cudaSuccess)                                                                    \
            return ::patchkv::fail((ctx), e_ == cudaErrorMemoryAllocation ? PATCHKV_E_NOMEM : PATCHKV_E_CUDA, \
                                   std::string(#expr) + ": " + cudaGetErrorString(e_));           \
    } while (0)

// Validates geometry + pool and fills the geometry / pool part of RestoreParams.
int fill_geometry(patchkv_ctx* ctx, const patchkv_geom* g, const patchkv_pool* pool, RestoreParams* p);
// cos / sin table of one session (double on the host, rounded once to fp32).
void build_rope_table(const patchkv_geom* g, int delta, float* cos_out, float* sin_out);
// Grows the pinned + device metadata arenas and the device staging ring of the host-resident entry points.
int ensure_host_workspace(patchkv_ctx* ctx, size_t meta_bytes, size_t slot_bytes);
// Launches the restore kernel for layers [layer_begin, layer_end) of the sessions already filled in p.
int launch_restore(patchkv_ctx* ctx, RestoreParams* p, cudaStream_t stream);
// The slot of work counters (two words of ctx->d_sched per slot) a self-scheduling launch on `stream` uses: one per
// stream the context has seen, one per launch captured into a graph.  The last CTA of a launch leaves its slot at zero.
int sched_slot(patchkv_ctx* ctx, cudaStream_t stream, bool capturing, int* slot);

}  // namespace patchkv
