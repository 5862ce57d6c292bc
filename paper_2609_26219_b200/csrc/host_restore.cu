// Restore from a CPU-resident checkpoint (Section II-C; Section V-A: CPU DRAM is the offload tier).
// Only the records of reused blocks cross the host link.  Per (session, layer) unit the planner merges the
// byte ranges of the reused records into a few large copies, issues them on a copy stream into one slot of
// a device staging ring at the same offsets they have in the layer payload (so the directory needs no
// rewriting), and launches the restore kernel for that unit on a decode stream as soon as the slot has
// landed.  Events order slot reuse; there is no device-side waiting.
#include <algorithm>

#include "common.cuh"

namespace patchkv {

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Grow the metadata arenas (device + pinned mirror) and the staging ring.  Growing synchronises the device.
int ensure_host_workspace(patchkv_ctx* ctx, size_t meta_bytes, size_t slot_bytes) {
    if (meta_bytes > ctx->meta_bytes) {
        PKV_CUDA(ctx, cudaDeviceSynchronize());
        if (ctx->d_meta) { cudaFree(ctx->d_meta); ctx->d_meta = nullptr; }
        if (ctx->h_meta) { cudaFreeHost(ctx->h_meta); ctx->h_meta = nullptr; ctx->h_meta_alias = nullptr; }
        ctx->meta_bytes = 0;
        PKV_CUDA(ctx, cudaMalloc(&ctx->d_meta, meta_bytes));
        PKV_CUDA(ctx, cudaHostAlloc(&ctx->h_meta, meta_bytes, cudaHostAllocMapped));
        void* a = nullptr;
        if (cudaHostGetDevicePointer(&a, ctx->h_meta, 0) != cudaSuccess) { cudaGetLastError(); a = nullptr; }
        ctx->h_meta_alias = static_cast<uint8_t*>(a);
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

namespace {

// A run of reused records that lie back to back in a layer payload (same-tag runs are contiguous in the checkpoint, so a
// run ends where a repaired block or the end of the tag's cluster interrupts it).
struct Run {
    uint64_t begin, end;        // byte range inside the layer payload
    int32_t first, count;       // its blocks: entries [first, first + count) of the unit's run-ordered block array
    bool staged;                // true: fetched by the copy engine into the staging slot; false: read over the link by the kernel
};

// Scratch of the per-unit planner, kept across units so that planning allocates nothing after the first unit.
struct UnitPlan {
    std::vector<Run> runs;
    std::vector<int32_t> run_of;    // per list position: its run, or -1
    std::vector<int32_t> blocks;    // reused blocks grouped by run
    std::vector<int32_t> stray;     // list entries that no run holds (out of range): left to the kernel, which latches the error
    std::vector<int32_t> by_size;   // run indices, shortest first
    uint64_t bytes = 0;
};

// Runs of one (session, layer), found in one pass over the reuse list: inside a tag's cluster the offsets rise with the
// block index, so a record either continues its tag's open run or starts a new one.
void plan_unit(const patchkv_session_host& s, int l, int nb, const uint64_t* rec_of, UnitPlan& u) {
    const int cnt = s.reuse_cnt[l];
    const uint8_t* tg = s.tags + (size_t)l * nb;
    const uint64_t* off = s.blk_off + (size_t)l * nb;
    const int32_t* list = s.reuse_idx + (size_t)l * nb;
    const uint64_t lbytes = s.layer_bytes[l];
    u.runs.clear(); u.stray.clear(); u.bytes = 0;
    u.run_of.assign(cnt, -1);
    int open_run[4] = {-1, -1, -1, -1};
    for (int r = 0; r < cnt; r++) {
        const int j = list[r];
        if (j < 0 || j >= nb) { u.stray.push_back(j); continue; }
        const int t = tg[j];
        const uint64_t rb = t <= PATCHKV_TAG_K4V4 ? rec_of[t] : 0, o = off[j];
        if (rb == 0 || o > lbytes || rb > lbytes - o) { u.stray.push_back(j); continue; }
        u.bytes += rb;
        int k = open_run[t];
        if (k >= 0 && u.runs[k].end == o) { u.runs[k].end = o + rb; u.runs[k].count++; }
        else { k = (int)u.runs.size(); u.runs.push_back({o, o + rb, 0, 1, true}); open_run[t] = k; }
        u.run_of[r] = k;
    }
    int32_t at = 0;
    for (auto& run : u.runs) { run.first = at; at += run.count; run.count = 0; }
    u.blocks.resize(at);
    for (int r = 0; r < cnt; r++) {
        const int k = u.run_of[r];
        if (k >= 0) u.blocks[u.runs[k].first + u.runs[k].count++] = list[r];
    }
}

}  // namespace

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
    base.grid_cap = 0;
    std::vector<RestoreParams> per(n_sessions, base);      // one single-session launch description per session
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, PATCHKV_E_CUDA, "cudaSetDevice failed");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int L = geom->n_layers, B = geom->block_tokens;
    const uint64_t elems = (uint64_t)B * geom->n_kv_heads * geom->head_dim;
    uint64_t rec_of[4];
    for (int t = 0; t < 4; t++) rec_of[t] = record_bytes(t, elems, geom->group);

    // ---- validate the sessions, size the metadata arena and the staging slots
    size_t slot_bytes = 0, meta = 0;
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
              + align_up((size_t)L * nb * 4, 256) * 2                  // reuse list(s)
              + align_up((size_t)L * 4, 256)                           // list lengths (or their upper bound)
              + align_up((size_t)L * 8, 256) * 3                       // layer_bytes, staged layer pointers, aliases
              + align_up((size_t)s.n_table * 4 + 4, 256);              // block_table
    }
    if (meta == 0) return PATCHKV_OK;

    // ---- how the records travel.  Staged: the copy engine fetches byte ranges into a device slot and the kernel decodes
    //      from there; a copy costs a few microseconds of engine time whatever its size, during which the link idles, so
    //      neighbouring ranges are merged across small gaps and the bytes in the gaps are wasted.  Direct: the kernel's
    //      own bulk copies read the pinned payload through its device alias; exactly the records cross the link, but
    //      reads issued by the SMs top out below the copy engine's rate.  Hybrid (the default) does both at once, layer
    //      by layer: the long runs of adjacent records go to the copy engine, one copy per run and not a byte wasted,
    //      while a small side launch reads the layer's short runs; each path's idle moments are the other's gain.
    const bool all_direct = (ctx->flags & PATCHKV_FLAG_HOST_DIRECT) != 0;
    bool staged_only = !all_direct && (ctx->flags & PATCHKV_FLAG_HOST_STAGED) != 0;
    // device aliases of the pinned layer payloads (direct and hybrid); without one a session cannot be read directly
    std::vector<std::vector<const void*>> alias(n_sessions);
    if (!staged_only) {
        bool have_alias = true;
        for (int i = 0; i < n_sessions && have_alias; i++) {
            alias[i].assign(L, nullptr);
            for (int l = 0; l < L && nbs[i] > 0; l++) {
                void* a = nullptr;
                if (sessions[i].layer_bytes[l] != 0 &&
                    cudaHostGetDevicePointer(&a, const_cast<void*>(sessions[i].layer_payload[l]), 0) != cudaSuccess) {
                    cudaGetLastError();
                    have_alias = false;
                    break;
                }
                alias[i][l] = a;
            }
        }
        if (!have_alias && all_direct) return fail(ctx, PATCHKV_E_INVALID, "session: pinned payload has no device alias (not mapped)");
        if (!have_alias) staged_only = true;
    }

    // A previous call may still be reading the metadata arenas and the ring: wait for it on the host.
    if (ctx->host_call_pending) {
        PKV_CUDA(ctx, cudaEventSynchronize(ctx->ev_done));
        ctx->host_call_pending = false;
    }
    rc = ensure_host_workspace(ctx, meta, all_direct ? 16 : std::max<size_t>(slot_bytes, 16));
    if (rc != PATCHKV_OK) return rc;
    const int n_slots = (int)ctx->slots.size();

    // ---- the internal streams start after whatever is already on the caller's stream
    PKV_CUDA(ctx, cudaEventRecord(ctx->ev_begin, stream));
    PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_begin, 0));
    PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->decode_stream, ctx->ev_begin, 0));
    PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->direct_stream, ctx->ev_begin, 0));

    // From here on work is enqueued on the internal streams.  Whatever happens below, the call leaves through
    // `join`, which makes the caller's stream wait for the internal streams and marks the context's arenas and ring
    // as in use, so that an error half-way never lets a later call (or the caller's stream) overtake queued work.
    auto join = [&](int code) -> int {
        cudaError_t e = cudaEventRecord(ctx->ev_begin, ctx->copy_stream);       // ev_begin has served its purpose above
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->decode_stream, ctx->ev_begin, 0);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_direct, ctx->direct_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->decode_stream, ctx->ev_direct, 0);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_done, ctx->decode_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, ctx->ev_done, 0);
        if (e == cudaSuccess) ctx->host_call_pending = true;
        else {                                                                   // cannot order it: drain it here
            cudaGetLastError();
            cudaStreamSynchronize(ctx->copy_stream);
            cudaStreamSynchronize(ctx->direct_stream);
            cudaStreamSynchronize(ctx->decode_stream);
            if (code == PATCHKV_OK) code = fail(ctx, PATCHKV_E_CUDA, std::string("restore_from_host: ") + cudaGetErrorString(e));
        }
        return code;
    };
    auto enqueue = [&]() -> int {
    // ---- metadata.  The directory (tags, offsets, block table, layer pointers) is staged in one pinned image and goes to
    //      the device in one copy.  The two reuse lists of a layer (staged blocks, directly read blocks) are written by
    //      the planner a few layers at a time, while earlier layers are already in flight, and follow in one small copy
    //      per group of layers; row l of the list area holds [staged blocks (nb) | direct blocks (nb)].
    size_t cur = 0;
    auto put = [&](const void* src, size_t bytes) -> size_t {
        const size_t at = cur;
        if (bytes) memcpy(ctx->h_meta + at, src, bytes);
        cur += align_up(bytes ? bytes : 1, 256);
        return at;
    };
    auto reserve = [&](size_t bytes) -> size_t {
        const size_t at = cur;
        cur += align_up(bytes ? bytes : 1, 256);
        return at;
    };
    std::vector<size_t> rows_at(n_sessions, 0);            // offset of each session's list area in the arenas
    std::vector<SessionDev> direct_dev(n_sessions);
    long long unit0 = 0;
    for (int i = 0; i < n_sessions; i++) {
        const patchkv_session_host& s = sessions[i];
        SessionDev& d = per[i].s[0];
        memset(&d, 0, sizeof(d));
        const int nb = nbs[i];
        d.n = s.n_suffix_tokens; d.nb = nb; d.list_nb = nb; d.delta = s.delta; d.dst_shift = s.dst_shift; d.n_table = s.n_table;
        direct_dev[i] = d;
        if (nb == 0) continue;
        d.tags = ctx->d_meta + put(s.tags, (size_t)L * nb);
        d.blk_off = reinterpret_cast<const unsigned long long*>(ctx->d_meta + put(s.blk_off, (size_t)L * nb * 8));
        d.layer_bytes = reinterpret_cast<const unsigned long long*>(ctx->d_meta + put(s.layer_bytes, (size_t)L * 8));
        d.block_table = reinterpret_cast<const int32_t*>(ctx->d_meta + put(s.block_table, (size_t)s.n_table * 4));
        std::vector<const void*> staged(L);
        for (int l = 0; l < L; l++) staged[l] = all_direct ? nullptr : ctx->slots[(unit0 + l) % n_slots].base;
        d.layer_payload = reinterpret_cast<const void* const*>(ctx->d_meta + put(staged.data(), (size_t)L * 8));
        const void* const* alias_ptrs = staged_only ? d.layer_payload
            : reinterpret_cast<const void* const*>(ctx->d_meta + put(alias[i].data(), (size_t)L * 8));
        build_rope_table(geom, s.delta, per[i].cs[0][0], per[i].cs[0][1]);
        if (all_direct) {       // the caller's list as it is, on the device with the rest
            d.reuse_idx = reinterpret_cast<const int32_t*>(ctx->d_meta + put(s.reuse_idx, (size_t)L * nb * 4));
            d.reuse_cnt = reinterpret_cast<const int32_t*>(ctx->d_meta + put(s.reuse_cnt, (size_t)L * 4));
            d.layer_payload = alias_ptrs;
            unit0 += L;
            continue;
        }
        // A launch of this path covers one layer and is told exactly how many entries its list has, so the per-layer
        // length the kernel compares against only has to be an upper bound.
        std::vector<int32_t> bound(L, nb);
        d.reuse_cnt = reinterpret_cast<const int32_t*>(ctx->d_meta + put(bound.data(), (size_t)L * 4));
        d.list_nb = 2 * nb;
        // the same session as the side launches see it: the other half of each row, the payload through its device alias
        direct_dev[i] = d;
        direct_dev[i].layer_payload = alias_ptrs;
        unit0 += L;
    }
    // the list areas lie behind everything that the first copy carries, so that copy never touches them
    const size_t directory_bytes = cur;
    for (int i = 0; i < n_sessions && !all_direct; i++) {
        if (nbs[i] == 0) continue;
        rows_at[i] = reserve((size_t)L * 2 * nbs[i] * 4);
        per[i].s[0].reuse_idx = reinterpret_cast<const int32_t*>(ctx->d_meta + rows_at[i]);
        direct_dev[i].reuse_idx = per[i].s[0].reuse_idx + nbs[i];
    }
    PKV_CUDA(ctx, cudaMemcpyAsync(ctx->d_meta, ctx->h_meta, directory_bytes, cudaMemcpyHostToDevice, ctx->decode_stream));
    PKV_CUDA(ctx, cudaEventRecord(ctx->ev_direct, ctx->decode_stream));            // the side launches need the directory too
    PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->direct_stream, ctx->ev_direct, 0));

    patchkv_restore_stats st;
    memset(&st, 0, sizeof(st));
    st.struct_size = sizeof(st);
    if (all_direct) {
        // one launch over every session and layer; exactly the reused records cross the link, pulled by the kernel
        RestoreParams& q = base;
        q.n_sessions = n_sessions; q.layer_begin = 0; q.layer_end = L; q.grid_cap = 0;
        long long items = 0;
        for (int i = 0; i < n_sessions; i++) {
            q.s[i] = per[i].s[0];
            memcpy(q.cs[i], per[i].cs[0], sizeof(q.cs[i]));
            q.s[i].item_begin = (int32_t)items;
            items += (long long)nbs[i] * L;
            if (nbs[i] == 0) q.s[i].list_nb = 1;
            if (items > 0x7fff0000LL) return fail(ctx, PATCHKV_E_UNSUPPORTED, "restore_from_host: too many work items");
            const patchkv_session_host& s = sessions[i];
            for (int l = 0; l < L && nbs[i] > 0; l++)
                for (int r = 0; r < s.reuse_cnt[l]; r++) {
                    const int j = s.reuse_idx[(size_t)l * nbs[i] + r];
                    if (j < 0 || j >= nbs[i]) continue;
                    const int t = s.tags[(size_t)l * nbs[i] + j];
                    if (t > PATCHKV_TAG_K4V4) continue;
                    st.bytes_useful += rec_of[t];
                    st.n_block_layers++;
                }
        }
        st.bytes_copied = st.bytes_direct = st.bytes_useful;
        q.total_items = (int32_t)items;
        rc = launch_restore(ctx, &q, ctx->decode_stream);
        if (rc != PATCHKV_OK) return rc;
        if (stats) *stats = st;
        return PATCHKV_OK;
    }

    // ---- one (session, layer) unit after the other, planned a few layers at a time so that the planner works while
    //      earlier layers are in flight: plan, send the group's lists, then per layer hand the copies to the engine and
    //      launch the decoders
    constexpr int kGroup = 4;
    UnitPlan plans[kGroup];
    std::vector<const Run*> order;
    const uint64_t merge_gap = staged_only ? ctx->merge_gap : 0;
    long long unit = 0;
    for (int i = 0; i < n_sessions; i++) {
        const patchkv_session_host& s = sessions[i];
        const int nb = nbs[i];
        if (nb == 0) continue;
        for (int l0 = 0; l0 < L;) {
            const int l1 = std::min(L, l0 + (unit == 0 ? 1 : kGroup));        // the very first group is one layer: start soon
            int32_t n_s[kGroup], n_d[kGroup];
            for (int l = l0; l < l1; l++) {
                UnitPlan& u = plans[l - l0];
                plan_unit(s, l, nb, rec_of, u);
                // The split.  While both paths have work they share the link about evenly, and whenever the engine sits
                // between two copies the side launch has the link to itself; the layer is done soonest when the two finish
                // together, i.e. when the side launch reads half of the bytes plus what fits into the engine's pauses.
                // The shortest runs go first (fewest copies left for the engine).  A side launch that falls behind only
                // costs its lower rate on the remainder; an engine left alone pays a pause per copy, so err high.
                for (auto& run : u.runs) run.staged = true;
                if (!staged_only) {
                    u.by_size.resize(u.runs.size());
                    for (size_t k = 0; k < u.runs.size(); k++) u.by_size[k] = (int32_t)k;
                    std::sort(u.by_size.begin(), u.by_size.end(), [&](int32_t a, int32_t b) {
                        return u.runs[a].end - u.runs[a].begin < u.runs[b].end - u.runs[b].begin; });
                    uint64_t got = 0, left = u.runs.size();
                    for (int32_t k : u.by_size) {
                        // (a run goes only if that brings the side launch's share closer to the target: a layer that
                        // is one long run stays with the engine whole)
                        const uint64_t bytes = u.runs[k].end - u.runs[k].begin;
                        if (got + bytes / 2 > u.bytes / 100 * ctx->direct_percent + left * ctx->pause_fill_bytes) break;
                        u.runs[k].staged = false;
                        got += bytes;
                        left--;
                    }
                }
                int32_t* ls = reinterpret_cast<int32_t*>(ctx->h_meta + rows_at[i]) + (size_t)l * 2 * nb;
                int32_t* ld = ls + nb;
                int32_t a = 0, b = 0;
                for (const auto& run : u.runs) {
                    memcpy(run.staged ? ls + a : ld + b, u.blocks.data() + run.first, (size_t)run.count * 4);
                    (run.staged ? a : b) += run.count;
                    if (!run.staged) st.bytes_direct += run.end - run.begin;
                }
                for (int32_t j : u.stray) ls[a++] = j;                    // the staged launch latches the error
                n_s[l - l0] = a; n_d[l - l0] = b;
                st.bytes_useful += u.bytes;
                st.n_block_layers += u.blocks.size();
            }
            const size_t at = rows_at[i] + (size_t)l0 * 2 * nb * 4;
            // (on the copy stream, ahead of the group's payload: both kernels of a layer start behind an event of that
            // stream, and a copy that had to wait for a kernel would hold up the engine's queue)
            PKV_CUDA(ctx, cudaMemcpyAsync(ctx->d_meta + at, ctx->h_meta + at, (size_t)(l1 - l0) * 2 * nb * 4,
                                          cudaMemcpyHostToDevice, ctx->copy_stream));
            for (int l = l0; l < l1; l++, unit++) {
                const UnitPlan& u = plans[l - l0];
                Staging& slot = ctx->slots[unit % n_slots];
                if (n_d[l - l0] > 0) {
                    // this layer's short runs: a small side launch that reads them over the link while the copy engine
                    // works on the layer's long runs (it starts when the copy stream reaches the layer)
                    static thread_local RestoreParams qd;
                    qd = per[i];
                    qd.s[0] = direct_dev[i];
                    qd.layer_begin = l; qd.layer_end = l + 1; qd.total_items = n_d[l - l0];
                    qd.grid_cap = ctx->direct_ctas;
                    PKV_CUDA(ctx, cudaEventRecord(ctx->ev_direct, ctx->copy_stream));
                    PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->direct_stream, ctx->ev_direct, 0));
                    rc = launch_restore(ctx, &qd, ctx->direct_stream);
                    if (rc != PATCHKV_OK) return rc;
                }
                if (n_s[l - l0] == 0) continue;
                // copies of this layer's staged runs, in ascending offset
                order.clear();
                for (const auto& run : u.runs) if (run.staged) order.push_back(&run);
                std::sort(order.begin(), order.end(), [](const Run* a, const Run* b) { return a->begin < b->begin; });
                if (unit >= n_slots) PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, slot.freed, 0));
                const uint8_t* src = static_cast<const uint8_t*>(s.layer_payload[l]);
                uint8_t* dst = static_cast<uint8_t*>(slot.base);
                for (size_t k = 0; k < order.size();) {
                    uint64_t b = order[k]->begin, e = order[k]->end;
                    size_t k2 = k + 1;
                    while (k2 < order.size() && order[k2]->begin <= e + merge_gap) { e = std::max(e, order[k2]->end); k2++; }
                    PKV_CUDA(ctx, cudaMemcpyAsync(dst + b, src + b, e - b, cudaMemcpyHostToDevice, ctx->copy_stream));
                    st.n_copies++;
                    st.bytes_copied += e - b;
                    k = k2;
                }
                PKV_CUDA(ctx, cudaEventRecord(slot.copied, ctx->copy_stream));
                PKV_CUDA(ctx, cudaStreamWaitEvent(ctx->decode_stream, slot.copied, 0));
                // one launch: the staged blocks of layer l of session i
                RestoreParams& q = per[i];
                q.layer_begin = l; q.layer_end = l + 1; q.total_items = n_s[l - l0];
                rc = launch_restore(ctx, &q, ctx->decode_stream);
                if (rc != PATCHKV_OK) return rc;
                PKV_CUDA(ctx, cudaEventRecord(slot.freed, ctx->decode_stream));
            }
            l0 = l1;
        }
    }
    st.bytes_copied += st.bytes_direct;
    if (stats) *stats = st;
    return PATCHKV_OK;
    };
    // ---- the caller's stream continues only after copy, decode and the side launches have drained
    return join(enqueue());
}
