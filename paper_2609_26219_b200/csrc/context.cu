// Context life cycle, error text and the device status word.
#include "common.cuh"

using namespace patchkv;

extern "C" int patchkv_create(patchkv_ctx** out, const patchkv_config* cfg) {
    if (!out || !cfg || cfg->struct_size != sizeof(patchkv_config)) return PATCHKV_E_INVALID;
    *out = nullptr;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cfg->device < 0 || cfg->device >= n_dev) return PATCHKV_E_CUDA;
    DeviceGuard guard(cfg->device);
    if (!guard.ok) return PATCHKV_E_CUDA;
    patchkv_ctx* ctx = new patchkv_ctx();
    ctx->device = cfg->device;
    ctx->staging_slots = cfg->staging_slots > 0 ? cfg->staging_slots : 4;
    if (ctx->staging_slots > 64) ctx->staging_slots = 64;
    ctx->flags = cfg->flags;
    ctx->merge_gap = cfg->merge_gap_bytes == UINT64_MAX ? 128 * 1024 : cfg->merge_gap_bytes;
    bool ok = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, cfg->device) == cudaSuccess;
    ok = ok && cudaDeviceGetAttribute(&ctx->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, cfg->device) == cudaSuccess;
    ok = ok && cudaDeviceGetAttribute(&ctx->smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, cfg->device) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&ctx->decode_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&ctx->direct_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&ctx->ev_direct, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&ctx->ev_begin, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&ctx->ev_done, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_status, sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMemset(ctx->d_status, 0, sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->d_sched, 2 * kSchedSlots * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMemset(ctx->d_sched, 0, 2 * kSchedSlots * sizeof(int32_t)) == cudaSuccess;
    if (!ok) {
        patchkv_destroy(ctx);
        return PATCHKV_E_CUDA;
    }
    *out = ctx;
    return PATCHKV_OK;
}

extern "C" int patchkv_destroy(patchkv_ctx* ctx) {
    if (!ctx) return PATCHKV_OK;
    {
        DeviceGuard guard(ctx->device);
        cudaDeviceSynchronize();
        for (auto& s : ctx->slots) {
            if (s.base) cudaFree(s.base);
            if (s.copied) cudaEventDestroy(s.copied);
            if (s.freed) cudaEventDestroy(s.freed);
        }
        if (ctx->d_meta) cudaFree(ctx->d_meta);
        if (ctx->h_meta) cudaFreeHost(ctx->h_meta);
        if (ctx->d_mass_ws) cudaFree(ctx->d_mass_ws);
        if (ctx->d_status) cudaFree(ctx->d_status);
        if (ctx->d_sched) cudaFree(ctx->d_sched);
        if (ctx->ev_begin) cudaEventDestroy(ctx->ev_begin);
        if (ctx->ev_done) cudaEventDestroy(ctx->ev_done);
        if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
        if (ctx->decode_stream) cudaStreamDestroy(ctx->decode_stream);
        if (ctx->direct_stream) cudaStreamDestroy(ctx->direct_stream);
        if (ctx->ev_direct) cudaEventDestroy(ctx->ev_direct);
    }
    delete ctx;
    return PATCHKV_OK;
}

extern "C" int patchkv_last_error(patchkv_ctx* ctx, char* buf, size_t n) {
    if (!ctx || !buf || n == 0) return PATCHKV_E_INVALID;
    std::lock_guard<std::mutex> lock(ctx->mu);
    strncpy(buf, ctx->last_error.c_str(), n - 1);
    buf[n - 1] = '\0';
    return PATCHKV_OK;
}

extern "C" int patchkv_query_status(patchkv_ctx* ctx, int* device_status) {
    if (!ctx || !device_status) return PATCHKV_E_INVALID;
    std::lock_guard<std::mutex> lock(ctx->mu);
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, PATCHKV_E_CUDA, "cudaSetDevice failed");
    PKV_CUDA(ctx, cudaDeviceSynchronize());
    int32_t v = 0;
    PKV_CUDA(ctx, cudaMemcpy(&v, ctx->d_status, sizeof(v), cudaMemcpyDeviceToHost));
    PKV_CUDA(ctx, cudaMemset(ctx->d_status, 0, sizeof(v)));
    *device_status = v;
    return PATCHKV_OK;
}

// A wait that nothing will ever satisfy, with a short limit: the same helper the pipeline kernels wait with has to give
// up, raise the abort flag and let the kernel report PATCHKV_E_TIMEOUT instead of spinning.
namespace patchkv {
__global__ void bounded_wait_selftest_kernel(uint32_t limit, int32_t* status) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const bool ok = mbar_wait(&bar, 0, &abort_flag, limit);       // no thread arrives on `bar`
    if (!__all_sync(0xFFFFFFFFu, ok) && (threadIdx.x & 31) == 0 && abort_flag)
        atomicCAS(status, 0, (int)PATCHKV_E_TIMEOUT);
}
}  // namespace patchkv

extern "C" int patchkv_selftest_bounded_wait(patchkv_ctx* ctx, uint32_t max_polls, void* stream) {
    if (!ctx) return PATCHKV_E_INVALID;
    std::lock_guard<std::mutex> lock(ctx->mu);
    if (max_polls == 0 || max_polls > (1u << 20)) return fail(ctx, PATCHKV_E_INVALID, "selftest: max_polls must be 1 .. 2^20");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, PATCHKV_E_CUDA, "cudaSetDevice failed");
    patchkv::bounded_wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(max_polls, ctx->d_status);
    PKV_CUDA(ctx, cudaGetLastError());
    return PATCHKV_OK;
}

extern "C" int patchkv_selftest_stall_next_launch(patchkv_ctx* ctx, int32_t after_units, uint32_t max_polls) {
    if (!ctx) return PATCHKV_E_INVALID;
    std::lock_guard<std::mutex> lock(ctx->mu);
    if (after_units < 0 || max_polls == 0 || max_polls > (1u << 20))
        return fail(ctx, PATCHKV_E_INVALID, "selftest: after_units >= 0, max_polls 1 .. 2^20");
    ctx->selftest_stall_after = after_units;
    ctx->selftest_wait_limit = max_polls;
    return PATCHKV_OK;
}

extern "C" uint64_t patchkv_record_bytes(int tag, int block_tokens, int n_kv_heads, int head_dim, int group) {
    if (block_tokens <= 0 || n_kv_heads <= 0 || head_dim <= 0 || group <= 0) return 0;
    return record_bytes(tag, (uint64_t)block_tokens * n_kv_heads * head_dim, group);
}
