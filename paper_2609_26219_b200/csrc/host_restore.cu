// Restore from a CPU-resident checkpoint (Section II-C; Section V-A: CPU DRAM is the offload tier).
// Only the records of reused blocks cross the host link.  Per (session, layer) unit the planner merges the
// byte ranges of the reused records into a few large copies, issues them on a copy stream into one slot of
// a device staging ring at the same offsets they have in the layer payload (so the directory needs no
// rewriting), and launches the restore kernel for that unit on a decode stream as soon as the slot has
// landed.  Events order slot reuse; there is no device-side waiting.
#include <algorithm>

#include "common.cuh"

namespace patchkv {

struct Range { uint64_t begin, end; };

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Grow the metadata arenas (device + pinned mirror) and the staging ring.  Growing synchronises the device.
int ensure_host_workspace(patchkv_ctx* ctx, size_t meta_bytes, size_t slot_bytes) {
    if (meta_bytes > ctx->meta_bytes) {
        PKV_CUDA(ctx, cudaDeviceSynchronize());
        if (ctx->d_meta) { cudaFree(ctx->d_meta); ctx->d_meta = nullptr; }
        if (ctx->h_meta) { cudaFreeHost(ctx->h_meta); ctx->h_meta = nullptr; }
        ctx->meta_bytes = 0;
        PKV_CUDA(ctx, cudaMalloc(&ctx->d_meta, meta_bytes));
        PKV_CUDA(ctx, cudaHostAlloc(&ctx->h_meta, meta_bytes, cudaHostAllocDefault));
        ctx->meta_bytes = meta_bytes;
    }
    if (ctx->slots.size() != (size_t)ctx->staging_slots) {
        ctx->slots.resize(ctx->staging_slots);
        for (auto& s : ctx->slots) {
            if (!s.copied) PKV_CUDA(ctx, cudaEventCreateWithFlags(&s.copied, cudaEventDisableTiming));
            if (!s.freed) PKV_CUDA(ctx, cudaEventCreateWithFlags(&s.freed, cudaEventDisableTiming));
        }
    }
    bool grow = false;
    for (auto& s : ctx->slots) grow = grow || s.bytes < slot_bytes;
    if (grow) {
        PKV_CUDA(ctx, cudaDeviceSynchronize());
        const size_t want = align_up(slot_bytes + slot_bytes / 8, 1 << 20);
        for (auto& s : ctx->slots) {
            if (s.base) { cudaFree(s.base); s.base = nullptr; s.bytes = 0; }
            PKV_CUDA(ctx, cudaMalloc(&s.base, want));
            s.bytes = want;
        }
    }
    return PATCHKV_OK;
}

}  // namespace patchkv

using namespace patchkv;

extern "C" int patchkv_restore_from_host(patchkv_ctx* ctx, const patchkv_geom* geom, const patchkv_pool* pool,
                                         const patchkv_session_host* sessions, int n_sessions, void* stream_,
                                         patchkv_restore_stats* stats) {
    if (!ctx) return PATCHKV_E_INVALID;
    std::lock_guard<std::mutex> lock(ctx->mu);
    if (n_sessions < 0 || n_sessions > PATCHKV_MAX_SESSIONS || (n_sessions > 0 && !sessions))
        return fail(ctx, PATCHKV_E_INVALID, "restore_from_host: n_sessions must be 0..PATCHKV_MAX_SESSIONS");
    if (stats && stats->struct_size != sizeof(patchkv_restore_stats))
        return fail(ctx, PATCHKV_E_INVALID, "restore_from_host: stats struct_size mismatch");
    static thread_local RestoreParams base;
    int rc = fill_geometry(ctx, geom, pool, &base);
    if (rc != PATCHKV_OK) return rc;
    base.n_sessions = 1;
    std::vector<RestoreParams> per(n_sessions, base);      // one single-session launch description per session
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, PATCHKV_E_CUDA, "cudaSetDevice failed");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int L = geom->n_layers, B = geom->block_tokens;
    const uint64_t elems = (uint64_t)B * geom->n_kv_heads * geom->head_dim;

    // ---- validate sessions, size the metadata arena and the staging slots
    size_t meta = 0, slot_bytes = 0;
    std::vector<int> nbs(n_sessions);
    for (int i = 0; i < n_sessions; i++) {
        const patchkv_session_host& s = sessions[i];
        if (s.struct_size != sizeof(patchkv_session_host)) return fail(ctx, PATCHKV_E_INVALID, "session: struct_size mismatch");
        if (s.n_suffix_tokens < 0 || s.dst_shift < 0 || s.dst_shift >= geom->page_tokens || s.n_table < 0)
            return fail(ctx, PATCHKV_E_INVALID, "session: n_suffix_tokens >= 0, 0 <= dst_shift < P, n_table >= 0");
        const int nb = (s.n_suffix_tokens + B - 1) / B;
        nbs[i] = nb;
        if (nb == 0) continue;
        if (!s.block_table || !s.tags || !s.blk_off || !s.layer_payload || !s.layer_bytes || !s.reuse_idx || !s.reuse_cnt)
            return fail(ctx, PATCHKV_E_INVALID, "session: null pointer");
        for (int l = 0; l < L; l++) {
            if (s.reuse_cnt[l] < 0 || s.reuse_cnt[l] > nb) return fail(ctx, PATCHKV_E_INVALID, "session: reuse_cnt out of range");
            if (s.layer_bytes[l] == 0) continue;
            if (!s.layer_payload[l] || (reinterpret_cast<uintptr_t>(s.layer_payload[l]) & 15u))
                return fail(ctx, PATCHKV_E_INVALID, "session: layer payload null or not 16-byte aligned");
            slot_bytes = std::max<size_t>(slot_bytes, s.layer_bytes[l]);
        }
        // the payload must be page-locked: an asynchronous copy from pageable memory would serialise
        cudaPointerAttributes attr;
        for (int l = 0; l < L; l += std::max(1, L - 1)) {           // first and last layer
            if (s.layer_bytes[l] == 0) continue;
            cudaError_t e = cudaPointerGetAttributes(&attr, s.layer_payload[l]);
            if (e != cudaSuccess || attr.type != cudaMemoryTypeHost) {
                cudaGetLastError();
                return fail(ctx, PATCHKV_E_INVALID, "session: layer payload is not pinned host memory");
            }
        }
        meta += align_up((size_t)L * nb, 256)                          // tags
              + align_up((size_t)L * nb * 8, 256)                      // blk_off
              + align_up((size_t)L * nb * 4, 256)                      // reuse_idx
              + align_up((size_t)L * 4, 256)                           // reuse_cnt
              + align_up((size_t)L * 8, 256) * 2                       // layer_bytes, staged layer pointers
              + align_up((size_t)s.n_table * 4 + 4, 256);              // block_table
    }
    if (meta == 0) return PATCHKV_OK;

    // A previous call may still be reading the metadata arenas and the ring: wait for it on the host.
    if (ctx->host_call_pending) {
        PKV_CUDA(ctx, cudaEventSynchronize(ctx->ev_done));
        ctx->host_call_pending = false;
    }
    const bool direct = (ctx->flags & PATCHKV_FLAG_HOST_DIRECT) != 0;
    rc = ensure_host_workspace(ctx, meta, direct ? 16 : std::max<size_t>(slot_bytes, 16));
    if (rc != PATCHKV_OK) return rc;
    const int n_slots = (int)ctx->slots.size();

    // ---- the internal streams start after whatever is already on the caller's stream
    PKV_CUDA(ctx, cudaEventRecord(ctx->ev_begin, stream));
    PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_begin, 0));
    PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->decode_stream, ctx->ev_begin, 0));

    // From here on work is enqueued on the internal streams.  Whatever happens below, the call leaves through
    // `join`, which makes the caller's stream wait for both internal streams and marks the context's arenas and ring
    // as in use, so that an error half-way never lets a later call (or the caller's stream) overtake queued work.
    auto join = [&](int code) -> int {
        cudaError_t e = cudaEventRecord(ctx->ev_begin, ctx->copy_stream);       // ev_begin has served its purpose above
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->decode_stream, ctx->ev_begin, 0);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_done, ctx->decode_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, ctx->ev_done, 0);
        if (e == cudaSuccess) ctx->host_call_pending = true;
        else {                                                                   // cannot order it: drain it here
            cudaGetLastError();
            cudaStreamSynchronize(ctx->copy_stream);
            cudaStreamSynchronize(ctx->decode_stream);
            if (code == PATCHKV_OK) code = fail(ctx, PATCHKV_E_CUDA, std::string("restore_from_host: ") + cudaGetErrorString(e));
        }
        return code;
    };
    auto enqueue = [&]() -> int {
    // ---- stage metadata: one pinned image, one copy; unit u (session-major, then layer) uses slot u % n_slots
    size_t cur = 0;
    auto put = [&](const void* src, size_t bytes) -> size_t {
        const size_t at = cur;
        if (bytes) memcpy(ctx->h_meta + at, src, bytes);
        cur += align_up(bytes ? bytes : 1, 256);
        return at;
    };
    long long unit0 = 0;
    for (int i = 0; i < n_sessions; i++) {
        const patchkv_session_host& s = sessions[i];
        SessionDev& d = per[i].s[0];
        memset(&d, 0, sizeof(d));
        const int nb = nbs[i];
        d.n = s.n_suffix_tokens; d.nb = nb; d.delta = s.delta; d.dst_shift = s.dst_shift; d.n_table = s.n_table;
        if (nb == 0) continue;
        d.tags = ctx->d_meta + put(s.tags, (size_t)L * nb);
        d.blk_off = reinterpret_cast<const unsigned long long*>(ctx->d_meta + put(s.blk_off, (size_t)L * nb * 8));
        d.reuse_idx = reinterpret_cast<const int32_t*>(ctx->d_meta + put(s.reuse_idx, (size_t)L * nb * 4));
        d.reuse_cnt = reinterpret_cast<const int32_t*>(ctx->d_meta + put(s.reuse_cnt, (size_t)L * 4));
        d.layer_bytes = reinterpret_cast<const unsigned long long*>(ctx->d_meta + put(s.layer_bytes, (size_t)L * 8));
        std::vector<const void*> staged(L);
        for (int l = 0; l < L; l++) {
            if (!direct) { staged[l] = ctx->slots[(unit0 + l) % n_slots].base; continue; }
            // zero-copy: the kernel's bulk copies read the pinned payload through its device alias
            void* alias = nullptr;
            if (s.layer_bytes[l] != 0 &&
                cudaHostGetDevicePointer(&alias, const_cast<void*>(s.layer_payload[l]), 0) != cudaSuccess) {
                cudaGetLastError();
                return fail(ctx, PATCHKV_E_INVALID, "session: pinned payload has no device alias (not mapped)");
            }
            staged[l] = alias;
        }
        d.layer_payload = reinterpret_cast<const void* const*>(ctx->d_meta + put(staged.data(), (size_t)L * 8));
        d.block_table = reinterpret_cast<const int32_t*>(ctx->d_meta + put(s.block_table, (size_t)s.n_table * 4));
        build_rope_table(geom, s.delta, per[i].cs[0][0], per[i].cs[0][1]);
        unit0 += L;
    }
    PKV_CUDA(ctx, cudaMemcpyAsync(ctx->d_meta, ctx->h_meta, cur, cudaMemcpyHostToDevice, ctx->decode_stream));

    patchkv_restore_stats st;
    memset(&st, 0, sizeof(st));
    st.struct_size = sizeof(st);
    if (direct) {
        // one launch over every session and layer; exactly the reused records cross the link, pulled by the kernel
        RestoreParams& q = base;
        q.n_sessions = n_sessions; q.layer_begin = 0; q.layer_end = L;
        long long items = 0;
        for (int i = 0; i < n_sessions; i++) {
            q.s[i] = per[i].s[0];
            memcpy(q.cs[i], per[i].cs[0], sizeof(q.cs[i]));
            q.s[i].item_begin = (int32_t)items;
            items += (long long)nbs[i] * L;
            if (items > 0x7fff0000LL) return fail(ctx, PATCHKV_E_UNSUPPORTED, "restore_from_host: too many work items");
            const patchkv_session_host& s = sessions[i];
            for (int l = 0; l < L && nbs[i] > 0; l++)
                for (int r = 0; r < s.reuse_cnt[l]; r++) {
                    const int j = s.reuse_idx[(size_t)l * nbs[i] + r];
                    if (j < 0 || j >= nbs[i]) continue;
                    st.bytes_useful += record_bytes(s.tags[(size_t)l * nbs[i] + j], elems, geom->group);
                    st.n_block_layers++;
                }
        }
        st.bytes_copied = st.bytes_useful;
        q.total_items = (int32_t)items;
        rc = launch_restore(ctx, &q, ctx->decode_stream);
        if (rc != PATCHKV_OK) return rc;
        if (stats) *stats = st;
        return PATCHKV_OK;
    }

    // ---- units
    std::vector<Range> ranges;
    long long unit = 0;
    for (int i = 0; i < n_sessions; i++) {
        const patchkv_session_host& s = sessions[i];
        const int nb = nbs[i];
        if (nb == 0) continue;
        for (int l = 0; l < L; l++, unit++) {
            Staging& slot = ctx->slots[unit % n_slots];
            // byte ranges of the reused records of this layer; out-of-range entries are left to the kernel,
            // which skips them and latches the error, so they are simply not fetched here
            ranges.clear();
            const int cnt = s.reuse_cnt[l];
            for (int r = 0; r < cnt; r++) {
                const int j = s.reuse_idx[(size_t)l * nb + r];
                if (j < 0 || j >= nb) continue;
                const uint64_t rec = record_bytes(s.tags[(size_t)l * nb + j], elems, geom->group);
                const uint64_t off = s.blk_off[(size_t)l * nb + j];
                if (rec == 0 || off > s.layer_bytes[l] || rec > s.layer_bytes[l] - off) continue;
                ranges.push_back({off, off + rec});
                st.bytes_useful += rec;
                st.n_block_layers++;
            }
            if (ranges.empty()) continue;
            std::sort(ranges.begin(), ranges.end(), [](const Range& a, const Range& b) { return a.begin < b.begin; });
            if (unit >= n_slots) PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, slot.freed, 0));
            const uint8_t* src = static_cast<const uint8_t*>(s.layer_payload[l]);
            uint8_t* dst = static_cast<uint8_t*>(slot.base);
            uint64_t b = ranges[0].begin, e = ranges[0].end;
            for (size_t k = 1; k <= ranges.size(); k++) {
                if (k < ranges.size() && ranges[k].begin <= e + ctx->merge_gap) {
                    e = std::max(e, ranges[k].end);
                    continue;
                }
                PKV_CUDA(ctx, cudaMemcpyAsync(dst + b, src + b, e - b, cudaMemcpyHostToDevice, ctx->copy_stream));
                st.n_copies++;
                st.bytes_copied += e - b;
                if (k < ranges.size()) { b = ranges[k].begin; e = ranges[k].end; }
            }
            PKV_CUDA(ctx, cudaEventRecord(slot.copied, ctx->copy_stream));
            PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->decode_stream, slot.copied, 0));
            // one launch: layer l of session i only
            RestoreParams& q = per[i];
            q.layer_begin = l; q.layer_end = l + 1; q.total_items = nb;
            rc = launch_restore(ctx, &q, ctx->decode_stream);
            if (rc != PATCHKV_OK) return rc;
            PKV_CUDA(ctx, cudaEventRecord(slot.freed, ctx->decode_stream));
        }
    }

    if (stats) *stats = st;
    return PATCHKV_OK;
    };
    // ---- the caller's stream continues only after copy and decode have drained
    return join(enqueue());
}
