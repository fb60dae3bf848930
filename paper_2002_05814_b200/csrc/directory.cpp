// The object table and the device-resident directory: rows, progress counters, published prefixes as the
// schedules see them, and the small per-launch resources (error records, timing events).
#include "context.h"

namespace hpl {

Object* find(hpl_ctx* c, int64_t id) {
    auto it = c->objects.find(id);
    return it == c->objects.end() ? nullptr : &it->second;
}

// Element prefix an object has published, as the schedules see it: of a Put object what was put (whole
// chunks); of a Reduce output (published when Reduce is called, Section 3.4.2) what its tree can already
// produce, i.e. the smallest prefix among its members once the tree is full.
uint64_t logical_ready_elems(hpl_ctx* c, int64_t oid) {
    Object* o = find(c, oid);
    if (!o) return 0;
    if (o->kind == OBJ_TARGET) {
        auto it = c->reduce_of_target.find(oid);
        if (it == c->reduce_of_target.end()) return 0;
        ReduceTreeSchedule& s = *c->reduces.at(it->second).sched;
        if (!s.full()) return 0;
        uint64_t m = object_elems(*o);
        for (int p = 0; p < s.k(); ++p) m = std::min(m, logical_ready_elems(c, s.object_at(p)));
        return m;
    }
    if (o->ready_bytes >= o->bytes) return object_elems(*o);
    return (uint64_t)published_chunks(c, *o) * object_chunk_elems(c, *o);
}

// The same prefix counted in the object's own chunks (chunk_bytes of its own dtype) ...
int64_t logical_delivered(hpl_ctx* c, int64_t oid) {
    Object* o = find(c, oid);
    if (!o) return 0;
    const uint64_t n = logical_ready_elems(c, oid);
    return n >= object_elems(*o) ? (int64_t)o->C : (int64_t)(n / object_chunk_elems(c, *o));
}

// ... and in the chunks of a Reduce (chunk_bytes of its input dtype: a bf16 Reduce works on twice as many
// elements per chunk as its fp32 output holds).
int64_t logical_delivered_in(hpl_ctx* c, int64_t oid, const ReduceOp& op) {
    Object* o = find(c, oid);
    if (!o) return 0;
    const uint64_t n = logical_ready_elems(c, oid);
    return n >= object_elems(*o) ? (int64_t)op.C : (int64_t)(n / op.chunk_elems);
}

// Elements of a Reduce output that earlier waves on the stream have produced (or will have, by stream order).
uint64_t produced_elems(hpl_ctx* c, const Object& o) {
    auto it = c->reduce_of_target.find(o.id);
    if (it == c->reduce_of_target.end()) return 0;
    const ReduceOp& op = c->reduces.at(it->second);
    if (op.merged.empty()) return 0;
    return std::min<uint64_t>((uint64_t)op.merged[0].full_prefix(op.n_ops(0)) * op.chunk_elems, op.elems);
}

int alloc_row(hpl_ctx* c, Object& o) {
    if (o.row >= 0) return HPL_OK;
    if (c->free_rows.empty()) return HPL_ERR_NOMEM;
    o.row = c->free_rows.back();
    c->free_rows.pop_back();
    DirRow& r = c->h_dir[o.row];
    r.ptr = (unsigned long long)(uintptr_t)o.ptr;
    r.bytes = o.bytes;
    r.n_chunks = o.C;
    // rows of library-produced copies are never polled: validity of their bytes is stream order
    r.ready_chunks = (o.kind == OBJ_PLAIN) ? 0u : o.C;
    r.dtype = (unsigned)o.dtype;
    r.owner = (unsigned)o.worker;
    // The row travels with the next flush (below), from a snapshot: the mirror itself keeps changing.
    if (c->device) c->dirty_rows.push_back(o.row);
    return HPL_OK;
}


// All rows changed on the host since the last flush go to the device in one copy per run of consecutive rows,
// from an immutable pinned snapshot, on the control stream: tiny copies only, which no polling kernel can hold
// up.  Kernels get the addresses of their operands with the launch, so a launch does not wait for these copies;
// only a wave that POLLS progress counters is ordered behind them (order_main_after_control).
int flush_directory(hpl_ctx* c) {
    if (!c->device) c->dirty_rows.clear();
    if (c->dirty_rows.empty()) return HPL_OK;
    std::sort(c->dirty_rows.begin(), c->dirty_rows.end());
    c->dirty_rows.erase(std::unique(c->dirty_rows.begin(), c->dirty_rows.end()), c->dirty_rows.end());
    size_t i = 0;
    while (i < c->dirty_rows.size()) {
        size_t j = i + 1;
        while (j < c->dirty_rows.size() && c->dirty_rows[j] == c->dirty_rows[j - 1] + 1) ++j;
        const uint32_t n = (uint32_t)(j - i);
        if (c->stage_cursor + n > kStageRows) {
            CUDA_TRY(cudaStreamSynchronize(c->ctl_stream));   // every earlier snapshot has been consumed
            c->stage_cursor = 0;
        }
        DirRow* snap = c->h_stage + c->stage_cursor;
        std::memcpy(snap, c->h_dir + c->dirty_rows[i], n * sizeof(DirRow));
        CUDA_TRY(cudaMemcpyAsync(c->d_dir + c->dirty_rows[i], snap, n * sizeof(DirRow), cudaMemcpyHostToDevice, c->ctl_stream));
        c->stage_cursor += n;
        i = j;
    }
    c->dirty_rows.clear();
    c->ctl_pending = true;
    return HPL_OK;
}

int order_main_after_control(hpl_ctx* c) {
    if (!c->ctl_pending) return HPL_OK;
    CUDA_TRY(cudaEventRecord(c->ctl_ev, c->ctl_stream));
    CUDA_TRY(cudaStreamWaitEvent(c->stream, c->ctl_ev, 0));
    c->ctl_pending = false;
    return HPL_OK;
}

// Publishes the chunk prefix of a put object in the device directory.  On the copy stream (chunks of a host
// object, behind the copy that brings them) it is a 4-byte update of the counter alone; otherwise the row is
// marked changed and travels with the next flush -- at once when kernels may be polling for it (plan-ahead).
int publish_counter(hpl_ctx* c, Object& o, uint32_t chunks, cudaStream_t s) {
    if (o.row < 0) return HPL_OK;
    c->h_dir[o.row].ready_chunks = chunks;   // the host mirror always holds the published value
    if (!c->device) return HPL_OK;
    if (s == c->copy_stream) {
        CUDA_TRY(cudaMemcpyAsync(&c->d_dir[o.row].ready_chunks, &c->h_iota[chunks], sizeof(uint32_t), cudaMemcpyHostToDevice, s));
        return HPL_OK;
    }
    c->dirty_rows.push_back(o.row);
    return c->cfg.plan_ahead ? flush_directory(c) : HPL_OK;
}

// The error record of the wave that is about to be launched.
DeviceStatus* next_wave_status(hpl_ctx* c) {
    const uint64_t idx = c->launch_seq - c->first_unchecked;
    c->wave_tag.push_back(c->batch_tag);
    ++c->launch_seq;
    return c->d_status + std::min<uint64_t>(idx, kStatusSlots - 1);
}

cudaEvent_t take_event(hpl_ctx* c) {
    if (!c->event_pool.empty()) {
        cudaEvent_t e = c->event_pool.back();
        c->event_pool.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

void collect_kernel_times(hpl_ctx* c) {   // call only after the stream has been waited for
    for (auto& t : c->timed) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, t.a, t.b) == cudaSuccess) {
            const uint64_t ns = (uint64_t)((double)ms * 1e6);
            if (t.kind == 0) c->stats.reduce_kernel_ns += ns; else c->stats.fanout_kernel_ns += ns;
        }
        c->event_pool.push_back(t.a);
        c->event_pool.push_back(t.b);
    }
    c->timed.clear();
}

// Arena blocks.  With debug_guard_bytes set (a testing aid: compute-sanitizer is not always available) every
// block is followed by a canary the library never writes; it is checked when the block is released and by
// hpl_check_guards, so that a kernel that runs past a target, a partial result or a store copy is noticed.
constexpr int kGuardPattern = 0xC5;

// Memory pressure (Section 6 of the paper: the copy made by Put is pinned until Delete, other copies may be evicted
// least recently used first).  What this store keeps beyond the pinned copies -- sources, Reduce outputs -- are the
// partial results of tree nodes: they can always be made again from the pinned sources.  When the arena is full the
// least recently used ones are dropped, except those of the Reduce that is being planned and those the current
// planning pass has already put into a task.  Returns whether anything was freed.
static bool evict_partial_results(hpl_ctx* c, uint64_t need) {
    if (c->world > 1) return false;
    std::vector<Object*> cand;
    for (auto& kv : c->objects) {
        Object& o = kv.second;
        if (o.kind == OBJ_PARTIAL && o.ptr && o.op_key != c->planning_target && o.last_pass != c->plan_pass) cand.push_back(&o);
    }
    if (cand.empty()) return false;
    std::sort(cand.begin(), cand.end(), [](Object* a, Object* b) { return a->last_use < b->last_use; });
    if (c->device) {   // enqueued work may still read them
        cudaStreamSynchronize(c->ctl_stream);
        cudaStreamSynchronize(c->copy_stream);
        cudaStreamSynchronize(c->stream);
    }
    uint64_t freed = 0;
    for (Object* o : cand) {
        auto it = c->reduce_of_target.find(o->op_key);
        if (it != c->reduce_of_target.end()) {
            ReduceOp& op = c->reduces.at(it->second);
            if (o->pos >= 0 && o->pos < (int)op.partial_key.size() && op.partial_key[o->pos] == o->id) {
                op.partial_key[o->pos] = 0;
                op.merged[o->pos].clear();    // what the buffer held is gone; what ancestors merged from it stands
            }
        }
        freed += o->bytes;
        const int64_t id = o->id;
        release_object_memory(c, *o);
        c->objects.erase(id);
        c->stats.evictions++;
        if (freed >= need) break;
    }
    return true;
}

Arena& arena_of_rank(hpl_ctx* c, int home) { return (home < 0 || home == c->rank || c->world <= 1) ? c->arena : c->peer_arenas[home]; }

// `home`: the rank on whose GPU the block lives (worker-per-GPU mode; every rank makes the same allocations in the same
// order in its replica of that rank's allocator, so the offset is known everywhere).  -1 = this rank.
void* arena_alloc(hpl_ctx* c, uint64_t n, int home) {
    Arena& ar = arena_of_rank(c, home);
    const bool local = &ar == &c->arena;
    if (!c->guard_bytes || !c->device) {
        void* q = ar.alloc(n);
        while (!q && local && evict_partial_results(c, n)) q = ar.alloc(n);
        return q;
    }
    const uint64_t body = (n + kAlign - 1) / kAlign * kAlign;
    uint8_t* p = (uint8_t*)ar.alloc(body + c->guard_bytes);
    while (!p && local && evict_partial_results(c, body + c->guard_bytes)) p = (uint8_t*)ar.alloc(body + c->guard_bytes);
    if (!p || !local) return p;      // (a remote block's canary is its owner's to write and check)
    // from the first byte behind the object (the padding up to the block's alignment is canary too)
    if (cudaMemsetAsync(p + n, kGuardPattern, body - n + c->guard_bytes, c->stream) != cudaSuccess) {
        ar.release(p);
        return nullptr;
    }
    c->guards[p] = {n, body - n + c->guard_bytes};
    return p;
}

// Bytes of the block's canary that no longer hold the pattern (waits for the device).
uint64_t check_guard(hpl_ctx* c, void* block) {
    auto g = c->guards.find(block);
    if (g == c->guards.end()) return 0;
    std::vector<uint8_t> host(g->second.second);
    cudaStreamSynchronize(c->stream);
    if (cudaMemcpy(host.data(), (uint8_t*)block + g->second.first, host.size(), cudaMemcpyDeviceToHost) != cudaSuccess) return 1;
    uint64_t bad = 0;
    for (uint8_t b : host) bad += b != kGuardPattern;
    return bad;
}

void arena_release(hpl_ctx* c, void* p) {
    if (c->guard_bytes && c->device && c->guards.count(p)) {
        c->guard_violations += check_guard(c, p);
        c->guards.erase(p);
    }
    if (c->world > 1) {   // the block belongs to the allocator whose range holds it
        for (int r = 0; r < c->world; ++r) {
            Arena& ar = arena_of_rank(c, r);
            if ((uint8_t*)p >= ar.base && (uint8_t*)p < ar.base + ar.size) {
                ar.release(p);
                return;
            }
        }
    }
    c->arena.release(p);
}

void release_object_memory(hpl_ctx* c, Object& o) {
    if (o.lib_owned && o.ptr) arena_release(c, o.ptr);
    o.ptr = nullptr;
    if (o.row >= 0) c->free_rows.push_back(o.row);
    o.row = -1;
}

}  // namespace hpl
