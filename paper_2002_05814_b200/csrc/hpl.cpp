// The C ABI (include/hpl.h): event handling, progress and waits.  The object table and device directory
// are in directory.cpp, the planners in plan_reduce.cpp and plan_bcast.cpp, the schedule builders in
// sched_reduce.cpp and sched_bcast.cpp, the kernels in kernels.cu.
//
// Division of labour (arXiv 2002.05814, Section 3): the schedule builders (sched_reduce.*,
// sched_bcast.*) decide WHO combines / forwards WHAT, as a function of the event timeline only.
// The planners decide HOW the pending part of those schedules is executed on the GPU right
// now: which subtrees of a reduce tree are complete for which chunks (those are fused into one
// pass in registers), which partial results must be materialised, which receivers can be served
// from which copy.  Execution order is free as long as the association order of the tree is
// kept, so the bits do not depend on it.
#include "context.h"

#include <dlfcn.h>

#include <mutex>
#include <set>

using namespace hpl;

namespace {

int sync_and_check(hpl_ctx* c);
int progress(hpl_ctx* c);
int plan_levels(hpl_ctx* c);

// Small objects (Section 3.2 treats objects under 64 KB apart: for them latency, not bandwidth, is the cost).
// Their collectives do not get launches of their own: the tasks planned for them in one pass are gathered and
// packed into shared waves -- one launch serves many small collectives, and a batch of Gets waits once.  A task is
// placed in the stage after everything it reads from: the levels of its own collective, and the collectives
// whose output it consumes.  Polling tasks stay out (a wait that runs out voids the wave it is in).
struct SmallBatch {
    struct R { ReduceOp* op; std::vector<PlannedReduceTask> tasks; int base; };
    struct F { BcastOp* op; std::vector<PlannedFanout> tasks; int stage; };
    std::vector<R> r;
    std::vector<F> f;
    std::unordered_map<int64_t, int> end_stage;   // output id -> last stage that writes it in this batch
    bool empty() const { return r.empty() && f.empty(); }
};

int flush_small(hpl_ctx* c, SmallBatch& sb) {
    if (sb.empty()) return HPL_OK;
    int last = 0;
    for (auto& x : sb.r)
        for (auto& t : x.tasks) last = std::max(last, x.base + t.level);
    for (auto& x : sb.f) last = std::max(last, x.stage);
    for (int stage = 1; stage <= last; ++stage) {
        for (int bf = 0; bf < 2; ++bf) {
            std::vector<std::pair<ReduceOp*, PlannedReduceTask*>> g;
            for (auto& x : sb.r)
                if ((x.op->in_dtype == HPL_BF16) == (bf == 1))
                    for (auto& t : x.tasks)
                        if (x.base + t.level == stage) g.push_back({x.op, &t});
            int rc = launch_reduce_group(c, g, bf == 1);
            if (rc != HPL_OK) return rc;
        }
        std::vector<std::pair<BcastOp*, PlannedFanout>> g;
        for (auto& x : sb.f)
            if (x.stage == stage)
                for (auto& t : x.tasks) g.push_back({x.op, std::move(t)});
        int rc = launch_fanout_group(c, g);
        if (rc != HPL_OK) return rc;
    }
    sb = SmallBatch();
    return HPL_OK;
}

// Planning a collective failed (the arena is exhausted, a node is too wide for a task) after parts of the same pass
// had been noted as planned: nothing of that pass was launched, so its notes are taken back -- to the values before,
// the buffers were not touched -- and the caller may make room and ask again.
void rollback_pass(hpl_ctx* c, uint64_t tag) {
    for (auto it = c->journal.r.rbegin(); it != c->journal.r.rend(); ++it) {
        if (it->tag != tag) continue;
        auto f = c->reduce_of_target.find(it->target);
        if (f == c->reduce_of_target.end()) continue;
        ReduceOp& op = c->reduces.at(f->second);
        if (it->pos < (int)op.merged.size()) op.merged[it->pos].set(it->a, it->b, it->old_v);
    }
    for (auto it = c->journal.b.rbegin(); it != c->journal.b.rend(); ++it) {
        if (it->tag != tag) continue;
        auto f = c->bcast_of_src.find(it->src);
        if (f == c->bcast_of_src.end()) continue;
        BcastOp& op = c->bcasts.at(f->second);
        if (it->loc < (int)op.phys_have.size()) op.phys_have[it->loc] = it->old_have;
    }
    auto& jr = c->journal.r;
    jr.erase(std::remove_if(jr.begin(), jr.end(), [tag](const Journal::R& e) { return e.tag == tag; }), jr.end());
    auto& jb = c->journal.b;
    jb.erase(std::remove_if(jb.begin(), jb.end(), [tag](const Journal::B& e) { return e.tag == tag; }), jb.end());
}

// Worker-per-GPU mode: the plan of one pass, identical on every rank, is kept as dependency levels; nothing is
// launched here.  A task sits in the level after everything it reads: the levels of its own tree below it, the
// collectives whose output it consumes.  hpl_run_level releases one level at a time, each rank launching the tasks
// whose output (reduce) or source copy (fan-out) lives on its GPU; the caller puts a barrier between levels.
int plan_levels(hpl_ctx* c) {
    if (!c->levels.empty()) return HPL_OK;   // the previous plan has not been run to its end yet
    std::unordered_map<int64_t, int> end_level;   // output id -> last level that writes it in this plan
    auto level_at = [c](int l) -> hpl_ctx::Level& {
        if ((int)c->levels.size() < l) c->levels.resize(l);
        return c->levels[l - 1];
    };
    auto ri = c->reduces.begin();
    auto bi = c->bcasts.begin();
    while (ri != c->reduces.end() || bi != c->bcasts.end()) {
        const bool take_reduce = bi == c->bcasts.end() || (ri != c->reduces.end() && ri->first < bi->first);
        c->batch_tag = ++c->tag_counter;
        if (take_reduce) {
            ReduceOp& op = ri->second;
            std::vector<PlannedReduceTask> tasks;
            int rc = plan_reduce(c, op, tasks);
            if (rc != HPL_OK) {
                rollback_pass(c, c->batch_tag);
                return rc;
            }
            int base = 0, top = 0;
            for (int p = 0; p < op.sched->k(); ++p) {
                auto e = end_level.find(op.sched->object_at(p));
                if (e != end_level.end()) base = std::max(base, e->second);
            }
            // a task's chunk range is released in pieces, one level apart: while a tree level works on a piece, the
            // level above it works on the piece before (pipelining across the levels, Section 3.3).  Pieces are the
            // groups of `pipeline_chunks` chunks counted from chunk 0 of the OBJECT, not from the task's first chunk:
            // tasks of one tree cover different ranges, and a parent's piece must come after the child's same piece.
            const uint32_t g = c->cfg.pipeline_chunks > 0 ? (uint32_t)c->cfg.pipeline_chunks : ~0u;
            uint32_t first_group = ~0u;
            for (auto& t : tasks) first_group = std::min(first_group, t.a / g);
            for (auto& t : tasks) {
                for (uint32_t a = t.a; a < t.b;) {
                    const uint32_t group = a / g;
                    const uint32_t b = (g == ~0u || (uint64_t)(group + 1) * g >= t.b) ? t.b : (group + 1) * g;
                    PlannedReduceTask piece = t;
                    piece.a = a;
                    piece.b = b;
                    const int lvl = t.level + (int)(group - first_group);
                    top = std::max(top, lvl);
                    level_at(base + lvl).r.push_back({&op, std::move(piece)});
                    a = b;
                }
            }
            if (top) end_level[op.target] = base + top;
            ++ri;
        } else {
            BcastOp& op = bi->second;
            std::vector<PlannedFanout> tasks;
            int rc = plan_bcast(c, op, tasks);
            if (rc != HPL_OK) {
                rollback_pass(c, c->batch_tag);
                return rc;
            }
            auto e = end_level.find(op.src);
            const int lvl = (e == end_level.end() ? 0 : e->second);
            const uint32_t g = c->cfg.pipeline_chunks > 0 ? (uint32_t)c->cfg.pipeline_chunks : ~0u;
            uint32_t first_group = ~0u;
            for (auto& t : tasks) first_group = std::min(first_group, t.a / g);
            for (auto& t : tasks) {   // hop h of the plan one level after hop h - 1, a piece one level after the piece before
                for (uint32_t a = t.a; a < t.b;) {
                    const uint32_t group = a / g;
                    const uint32_t b = (g == ~0u || (uint64_t)(group + 1) * g >= t.b) ? t.b : (group + 1) * g;
                    PlannedFanout piece = t;
                    piece.a = a;
                    piece.b = b;
                    level_at(lvl + t.level + (int)(group - first_group)).f.push_back({&op, std::move(piece)});
                    a = b;
                }
            }
            ++bi;
        }
    }
    return HPL_OK;
}

int run_level(hpl_ctx* c) {
    if (c->levels.empty()) return HPL_OK;
    hpl_ctx::Level lv = std::move(c->levels.front());
    c->levels.erase(c->levels.begin());
    for (int bf = 0; bf < 2; ++bf) {
        std::vector<std::pair<ReduceOp*, PlannedReduceTask*>> g;
        for (auto& x : lv.r) {
            if ((x.first->in_dtype == HPL_BF16) != (bf == 1)) continue;
            Object* out = nullptr;
            int rc = ensure_partial_buffer(c, *x.first, x.second.pos, &out);
            if (rc != HPL_OK) return rc;
            if (out->home == c->rank) g.push_back({x.first, &x.second});   // owner computes
        }
        int rc = launch_reduce_group(c, g, bf == 1);
        if (rc != HPL_OK) return rc;
    }
    std::vector<std::pair<BcastOp*, PlannedFanout>> g;
    for (auto& x : lv.f) {
        const auto& locs = x.first->sched->locations();
        Object* from = x.second.loc == 0 ? find(c, x.first->src) : find(c, locs[x.second.loc].obj);
        if (from && from->home == c->rank) g.push_back(std::move(x));   // the holder of the copy pushes it to its receivers
    }
    return launch_fanout_group(c, g);
}

int progress(hpl_ctx* c) {
    ++c->plan_pass;
    // (a schedule-only context plans as well -- its planned tasks are counted, nothing is launched)
    {
        int rc = flush_directory(c);
        if (rc != HPL_OK) return rc;
    }
    if (c->copy_pending && !c->cfg.plan_ahead) {
        // host objects: their chunks become usable once the main stream is ordered after the copies
        CUDA_TRY(cudaEventRecord(c->copy_ev, c->copy_stream));
        CUDA_TRY(cudaStreamWaitEvent(c->stream, c->copy_ev, 0));
        c->copy_pending = false;
        for (auto& kv : c->objects)
            if (kv.second.async_counter) kv.second.landed = published_chunks(c, kv.second);
    }
    if (c->world > 1) return plan_levels(c);
    // collectives in creation order, so that one that consumes another's output (composed Reduce, reduce
    // followed by broadcast) is planned after its producer and launched behind it on the stream
    SmallBatch sb;
    auto ri = c->reduces.begin();
    auto bi = c->bcasts.begin();
    while (ri != c->reduces.end() || bi != c->bcasts.end()) {
        const bool take_reduce = bi == c->bcasts.end() || (ri != c->reduces.end() && ri->first < bi->first);
        c->batch_tag = ++c->tag_counter;
        if (take_reduce) {
            ReduceOp& op = ri->second;
            std::vector<PlannedReduceTask> tasks;
            int rc = plan_reduce(c, op, tasks);
            if (rc == HPL_ERR_NOMEM && c->device && (c->work_in_flight || !sb.empty())) {
                // The arena is full of partial results that this pass itself (or work still in flight) uses.  What was
                // planned so far runs to its end; after that those buffers may go, least recently used first, and this
                // Reduce is planned again, as a pass of its own.
                rollback_pass(c, c->batch_tag);
                int rc2 = flush_small(c, sb);
                if (rc2 == HPL_OK) rc2 = sync_and_check(c);
                // (a polling wave whose wait ran out has been voided by that call and is planned again by a later pass:
                // no reason to fail the event that happened to need the room)
                if (rc2 != HPL_OK && rc2 != HPL_ERR_TIMEOUT) return rc2;
                ++c->plan_pass;
                c->batch_tag = ++c->tag_counter;
                tasks.clear();
                rc = plan_reduce(c, op, tasks);
            }
            if (rc != HPL_OK) {   // what was planned before it runs all the same
                rollback_pass(c, c->batch_tag);
                flush_small(c, sb);
                return rc;
            }
            bool small = op.elems * 4 <= kSmallObjectBytes;
            for (auto& t : tasks) small = small && !t.poll;
            if (small && !tasks.empty()) {
                int base = 0, top = 0;
                for (int p = 0; p < op.sched->k(); ++p) {   // behind the collectives whose output is a member
                    auto e = sb.end_stage.find(op.sched->object_at(p));
                    if (e != sb.end_stage.end()) base = std::max(base, e->second);
                }
                for (auto& t : tasks) top = std::max(top, t.level);
                sb.end_stage[op.target] = base + top;
                sb.r.push_back({&op, std::move(tasks), base});
            } else if (!tasks.empty()) {
                // what was planned earlier is launched earlier.  (The tag of this planning pass stays as it was set
                // before planning: the journal entries made above carry it, and the waves launched below must too, or a
                // wait that runs out in one of them would not void them.)
                rc = flush_small(c, sb);
                if (rc != HPL_OK) return rc;
                rc = launch_reduce_tasks(c, op, tasks);
                if (rc != HPL_OK) return rc;
            }
            ++ri;
        } else {
            BcastOp& op = bi->second;
            std::vector<PlannedFanout> tasks;
            int rc = plan_bcast(c, op, tasks);
            if (rc != HPL_OK) {
                rollback_pass(c, c->batch_tag);
                flush_small(c, sb);
                return rc;
            }
            Object* src = find(c, op.src);
            bool small = src && src->bytes <= kSmallObjectBytes;
            for (auto& t : tasks) small = small && !t.poll;
            if (small && !tasks.empty()) {
                auto e = sb.end_stage.find(op.src);
                sb.f.push_back({&op, std::move(tasks), (e == sb.end_stage.end() ? 0 : e->second) + 1});
            } else if (!tasks.empty()) {
                rc = flush_small(c, sb);
                if (rc != HPL_OK) return rc;
                rc = launch_fanout_tasks(c, op, tasks);
                if (rc != HPL_OK) return rc;
            }
            ++bi;
        }
    }
    return flush_small(c, sb);
}

// A wave gave up.  Void: what its own planning pass had planned (tags in `failed`), whatever later passes planned
// for the same collectives (they may have continued in place from a buffer the wave left half updated), and whatever
// was planned since for collectives that consume their outputs, directly or not.  Collectives that have nothing to do
// with them keep their work: their waves ran to completion.  `everything`: the failed wave could not be told apart
// (more waves in flight than error records), so all passes from `from_tag` on are void.
void undo_journal(hpl_ctx* c, uint64_t from_tag, const std::set<uint64_t>& failed, bool everything) {
    std::set<int64_t> void_targets, void_srcs;
    for (auto& e : c->journal.r)
        if (everything ? e.tag >= from_tag : failed.count(e.tag) != 0) void_targets.insert(e.target);
    for (auto& e : c->journal.b)
        if (everything ? e.tag >= from_tag : failed.count(e.tag) != 0) void_srcs.insert(e.src);
    for (bool grew = true; grew;) {
        grew = false;
        for (auto& kv : c->reduces) {
            ReduceOp& op = kv.second;
            if (void_targets.count(op.target)) continue;
            for (int64_t sid : op.sched->sources())
                if (void_targets.count(sid)) {
                    void_targets.insert(op.target);
                    grew = true;
                    break;
                }
        }
    }
    for (auto& kv : c->bcasts)
        if (void_targets.count(kv.second.src)) void_srcs.insert(kv.second.src);
    for (auto& e : c->journal.r) {
        if (e.tag < from_tag || !void_targets.count(e.target)) continue;
        auto it = c->reduce_of_target.find(e.target);
        if (it == c->reduce_of_target.end()) continue;
        ReduceOp& op = c->reduces.at(it->second);
        // back to nothing, not to the earlier value: a task that gave up half way may have updated part of the
        // buffer in place, so what it held before is gone as well
        if (e.pos < (int)op.merged.size()) op.merged[e.pos].set(e.a, e.b, 0);
    }
    for (auto it = c->journal.b.rbegin(); it != c->journal.b.rend(); ++it) {
        if (it->tag < from_tag || !void_srcs.count(it->src)) continue;
        auto f = c->bcast_of_src.find(it->src);
        if (f == c->bcast_of_src.end()) continue;
        BcastOp& op = c->bcasts.at(f->second);
        if (it->loc < (int)op.phys_have.size()) op.phys_have[it->loc] = it->old_have;
    }
    c->journal.clear();   // everything in flight has been waited for: what was not voided is confirmed
}

int sync_and_check(hpl_ctx* c) {
    if (!c->device) {
        c->journal.clear();
        return HPL_OK;
    }
    if (c->copy_pending || c->ctl_unconfirmed) {
        CUDA_TRY(cudaStreamSynchronize(c->ctl_stream));
        CUDA_TRY(cudaStreamSynchronize(c->copy_stream));
        c->copy_pending = false;
        c->ctl_pending = false;
        c->ctl_unconfirmed = false;
        for (auto& kv : c->objects)
            if (kv.second.async_counter) kv.second.landed = published_chunks(c, kv.second);
    }
    if (!c->work_in_flight) {   // nothing of the library's is running: nothing to wait for
        c->journal.clear();
        return HPL_OK;
    }
    if (!c->polling_in_flight) {
        // no wave in flight waits on a counter, so no error record can have been written: nothing to read back
        CUDA_TRY(cudaStreamSynchronize(c->stream));
        c->work_in_flight = false;
        collect_kernel_times(c);
        c->first_unchecked = c->launch_seq;
        c->wave_tag.clear();
        c->journal.clear();
        return HPL_OK;
    }
    const uint32_t used = (uint32_t)std::min<uint64_t>(c->launch_seq - c->first_unchecked, kStatusSlots);
    CUDA_TRY(cudaMemcpyAsync(c->h_status, c->d_status, sizeof(DeviceStatus) * used, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    c->work_in_flight = false;
    collect_kernel_times(c);
    bool failed = false, ambiguous = false;
    uint64_t from_tag = ~0ull;
    std::set<uint64_t> failed_tags;
    for (uint32_t i = 0; i < used; ++i) {
        c->stats.device_waits += c->h_status[i].waits;
        if (!c->h_status[i].error) continue;
        if (c->h_status[i].error == 2) c->stats.bounds_errors++;   // (bounds-checking build) a tile was outside its object and was skipped
        failed = true;
        // the record in the last slot may stand for several waves: the earliest of them decides
        const uint64_t tag = c->wave_tag[i];
        from_tag = std::min(from_tag, tag);
        failed_tags.insert(tag);
        if (i == kStatusSlots - 1 && c->launch_seq - c->first_unchecked > kStatusSlots) ambiguous = true;
    }
    c->first_unchecked = c->launch_seq;
    c->wave_tag.clear();
    c->polling_in_flight = false;
    // the records are cleared behind everything launched so far; later launches are ordered after that
    CUDA_TRY(cudaMemsetAsync(c->d_status, 0, sizeof(DeviceStatus) * used, c->stream));
    if (failed) {
        c->stats.device_timeouts++;
        undo_journal(c, from_tag, failed_tags, ambiguous);
        return HPL_ERR_TIMEOUT;
    }
    c->journal.clear();
    return HPL_OK;
}

int after_event(hpl_ctx* c) { return c->cfg.eager ? progress(c) : HPL_OK; }

// After every event: a broadcast whose source is a Reduce output learns how far that output has got.
void refresh_composed(hpl_ctx* c) {
    for (uint64_t key : c->composed_bcasts) {   // only those: a Put must not cost time in proportion to all broadcasts
        BcastOp& op = c->bcasts.at(key);
        op.sched->source_progress((int64_t)c->now, logical_delivered(c, op.src));
    }
}

// The value of `target` changes (a member of its tree was replaced): whatever was computed from it is void.
void invalidate_consumers(hpl_ctx* c, int64_t target) {
    for (auto& kv : c->reduces) {
        ReduceOp& op = kv.second;
        if (!op.sched->has_source(target)) continue;
        for (auto& cs : op.merged) cs.clear();
        invalidate_consumers(c, op.target);
    }
    auto b = c->bcast_of_src.find(target);
    if (b != c->bcast_of_src.end()) {
        BcastOp& op = c->bcasts.at(b->second);
        std::fill(op.phys_have.begin(), op.phys_have.end(), 0);
    }
}

void notify_arrival(hpl_ctx* c, Object& o) {
    const int64_t id = o.id;
    o.consumers.for_each([c, id](uint64_t key) {   // in creation order
        auto r = c->reduces.find(key);
        if (r != c->reduces.end()) r->second.sched->arrive(id);
    });
}

int do_put_common(hpl_ctx* c, Object& o, uint64_t bytes, bool first) {
    o.ready_bytes = bytes;
    if (first) {
        o.arrived = true;
        o.t_arrival = (int64_t)c->now;
        notify_arrival(c, o);
    }
    auto b = c->bcast_of_src.find(o.id);
    if (b != c->bcast_of_src.end()) c->bcasts.at(b->second).sched->source_progress((int64_t)c->now, published_chunks(c, o));
    refresh_composed(c);
    return HPL_OK;
}

}  // namespace

// ================================================================================================ C ABI
extern "C" {

const char* hpl_strerror(int code) {
    switch (code) {
        case HPL_OK: return "ok";
        case HPL_ERR_INVALID: return "invalid argument";
        case HPL_ERR_NOT_FOUND: return "unknown object";
        case HPL_ERR_EXISTS: return "object id already exists";
        case HPL_ERR_TIMEOUT: return "not complete (bounded wait expired or inputs missing)";
        case HPL_ERR_INSUFFICIENT: return "no live source left";
        case HPL_ERR_FAILED_WORKER: return "owned by a failed worker";
        case HPL_ERR_CUDA: return "CUDA error or no device";
        case HPL_ERR_NOMEM: return "arena exhausted";
        default: return "unknown error";
    }
}

int hpl_init(const hpl_config* cfg, void* cuda_stream, hpl_ctx** out) {
    if (!cfg || !out) return HPL_ERR_INVALID;
    if (cfg->chunk_bytes == 0 || cfg->chunk_bytes % 16 || cfg->reduce_degree < 0 || cfg->bcast_degree < 1) return HPL_ERR_INVALID;
    if (cfg->reduce_degree == 0 && (cfg->model_latency_ns == 0 || cfg->model_bandwidth_bps == 0)) return HPL_ERR_INVALID;
    if (cfg->world_size > 1 && (cfg->rank < 0 || cfg->rank >= cfg->world_size || cfg->plan_ahead || cfg->eager)) return HPL_ERR_INVALID;
    hpl_ctx* c = new (std::nothrow) hpl_ctx();
    if (!c) return HPL_ERR_NOMEM;
    c->cfg = *cfg;
    if (cfg->world_size > 1) {
        c->rank = cfg->rank;
        c->world = cfg->world_size;
        c->rank_alive.assign(c->world, 1);
    }
    if (c->cfg.poll_budget_ns == 0) c->cfg.poll_budget_ns = 2000000000ull;
    c->tau = cfg->virt_chunk_ns ? cfg->virt_chunk_ns : std::max<uint64_t>(1, cfg->chunk_bytes * 1000000000ull / (64ull << 30));
    c->stream = (cudaStream_t)cuda_stream;
    if (cfg->arena) {
        const uint64_t need = sizeof(DirRow) * kMaxRows + sizeof(DeviceStatus) * kStatusSlots + 2 * kAlign;
        if (cfg->arena_bytes < need) {
            delete c;
            return HPL_ERR_NOMEM;
        }
        int dev = 0;
        cudaDeviceProp prop;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
            delete c;
            return HPL_ERR_CUDA;
        }
        c->n_sm = prop.multiProcessorCount;
        c->arena.init(cfg->arena, cfg->arena_bytes);
        c->d_dir = (DirRow*)c->arena.alloc(sizeof(DirRow) * kMaxRows);
        c->d_status = (DeviceStatus*)c->arena.alloc(sizeof(DeviceStatus) * kStatusSlots);
        bool ok = c->d_dir && c->d_status;
        ok = ok && cudaHostAlloc((void**)&c->h_dir, sizeof(DirRow) * kMaxRows, cudaHostAllocDefault) == cudaSuccess;
        ok = ok && cudaHostAlloc((void**)&c->h_status, sizeof(DeviceStatus) * kStatusSlots, cudaHostAllocDefault) == cudaSuccess;
        ok = ok && cudaHostAlloc((void**)&c->h_stage, sizeof(DirRow) * kStageRows, cudaHostAllocDefault) == cudaSuccess;
        ok = ok && cudaHostAlloc((void**)&c->h_iota, sizeof(uint32_t) * (kMaxChunks + 1), cudaHostAllocDefault) == cudaSuccess;
        ok = ok && cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
        ok = ok && cudaStreamCreateWithFlags(&c->ctl_stream, cudaStreamNonBlocking) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&c->copy_ev, cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&c->ctl_ev, cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaMemsetAsync(c->d_dir, 0, sizeof(DirRow) * kMaxRows, c->stream) == cudaSuccess;
        ok = ok && cudaMemsetAsync(c->d_status, 0, sizeof(DeviceStatus) * kStatusSlots, c->stream) == cudaSuccess;
        ok = ok && cudaStreamSynchronize(c->stream) == cudaSuccess;   // side streams must not overtake the clearing
        if (!ok) {
            if (c->h_dir) cudaFreeHost(c->h_dir);
            if (c->h_status) cudaFreeHost(c->h_status);
            if (c->h_stage) cudaFreeHost(c->h_stage);
            if (c->h_iota) cudaFreeHost(c->h_iota);
            if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
            if (c->ctl_stream) cudaStreamDestroy(c->ctl_stream);
            if (c->copy_ev) cudaEventDestroy(c->copy_ev);
            if (c->ctl_ev) cudaEventDestroy(c->ctl_ev);
            delete c;
            return HPL_ERR_CUDA;
        }
        c->guard_bytes = (cfg->debug_guard_bytes + kAlign - 1) / kAlign * kAlign;
        for (uint32_t i = 0; i <= kMaxChunks; ++i) c->h_iota[i] = i;
        for (int r = (int)kMaxRows - 1; r >= 0; --r) c->free_rows.push_back(r);
        c->device = true;
    } else {
        // schedule-only context: no device memory.  Addresses are handed out from a range that is never
        // dereferenced, so that the planners run exactly as they would with an arena.
        c->arena.init((void*)(uintptr_t)(1ull << 44), 1ull << 44);
        c->h_dir = (DirRow*)std::calloc(kMaxRows, sizeof(DirRow));
        if (!c->h_dir) {
            delete c;
            return HPL_ERR_NOMEM;
        }
        for (int r = (int)kMaxRows - 1; r >= 0; --r) c->free_rows.push_back(r);
        c->n_sm = 148;
    }
    if (c->world > 1) {
        // replicas of the other ranks' allocators: same size, same first allocations (directory, error records), so
        // that every later allocation lands at the same offset everywhere.  Their base addresses are set by
        // hpl_set_peer_arena; until then (and in a schedule-only context) a range that is never dereferenced stands in.
        c->peer_arenas.resize(c->world);
        for (int r = 0; r < c->world; ++r) {
            if (r == c->rank) continue;
            c->peer_arenas[r].init((void*)(uintptr_t)((1ull << 45) + ((uint64_t)r << 40)), c->arena.size);
            c->peer_arenas[r].alloc(sizeof(DirRow) * kMaxRows);
            c->peer_arenas[r].alloc(sizeof(DeviceStatus) * kStatusSlots);
        }
        if (!c->device) {   // the schedule-only arena takes the same two blocks, like a device one
            c->arena.alloc(sizeof(DirRow) * kMaxRows);
            c->arena.alloc(sizeof(DeviceStatus) * kStatusSlots);
        }
    }
    *out = c;
    return HPL_OK;
}

int hpl_shutdown(hpl_ctx* c) {
    if (!c) return HPL_ERR_INVALID;
    if (c->device) {
        cudaStreamSynchronize(c->ctl_stream);
        cudaStreamSynchronize(c->copy_stream);
        cudaStreamSynchronize(c->stream);
        collect_kernel_times(c);
        for (cudaEvent_t e : c->event_pool) cudaEventDestroy(e);
        cudaFreeHost(c->h_dir);
        cudaFreeHost(c->h_status);
        cudaFreeHost(c->h_stage);
        cudaFreeHost(c->h_iota);
        cudaStreamDestroy(c->copy_stream);
        cudaStreamDestroy(c->ctl_stream);
        cudaEventDestroy(c->copy_ev);
        cudaEventDestroy(c->ctl_ev);
    }
    if (!c->device) std::free(c->h_dir);
    delete c;
    return HPL_OK;
}

int hpl_advance(hpl_ctx* c, uint64_t t_ns) {
    if (!c || t_ns < c->now) return HPL_ERR_INVALID;
    c->now = t_ns;
    for (auto& kv : c->bcasts) kv.second.sched->advance((int64_t)t_ns);
    return HPL_OK;
}

int hpl_create(hpl_ctx* c, int64_t id, int32_t worker, uint64_t total_bytes, int32_t dtype) {
    if (!c || id < 0 || worker < 0 || (dtype != HPL_F32 && dtype != HPL_BF16)) return HPL_ERR_INVALID;
    if (total_bytes == 0 || total_bytes % elem_size(dtype)) return HPL_ERR_INVALID;
    if (c->objects.count(id)) return HPL_ERR_EXISTS;
    const uint64_t C = (total_bytes + c->cfg.chunk_bytes - 1) / c->cfg.chunk_bytes;
    if (C > kMaxChunks) return HPL_ERR_INVALID;
    Object o;
    o.id = id;
    o.worker = worker;
    o.bytes = total_bytes;
    o.dtype = dtype;
    o.C = (uint32_t)C;
    o.seq = c->seq++;
    c->objects.emplace(id, o);
    return HPL_OK;
}

static int put_checks(hpl_ctx* c, int64_t id, const void* buf, uint64_t bytes, Object** out) {
    if (!c || !buf) return HPL_ERR_INVALID;
    Object* o = find(c, id);
    if (!o) return HPL_ERR_NOT_FOUND;
    if (!o->alive) return HPL_ERR_FAILED_WORKER;
    if (o->kind != OBJ_PLAIN) return HPL_ERR_INVALID;
    if (bytes < o->ready_bytes || bytes > o->bytes) return HPL_ERR_INVALID;
    *out = o;
    return HPL_OK;
}

int hpl_put(hpl_ctx* c, int64_t id, const void* buf, uint64_t bytes) {
    Object* o = nullptr;
    int rc = put_checks(c, id, buf, bytes, &o);
    if (rc != HPL_OK) return rc;
    if ((uintptr_t)buf % 16) return HPL_ERR_INVALID;
    const bool first = !o->arrived;
    if (!first && (o->ptr != buf || o->from_host)) return HPL_ERR_INVALID;
    if (first) {
        o->ptr = const_cast<void*>(buf);
        o->home = c->world > 1 ? o->worker % c->world : 0;
        rc = alloc_row(c, *o);
        if (rc != HPL_OK) {
            o->ptr = nullptr;
            return rc;
        }
    }
    const uint32_t before = published_chunks(c, *o);
    do_put_common(c, *o, bytes, first);
    const uint32_t after = published_chunks(c, *o);
    if (c->device && c->cfg.plan_ahead) {
        // the counter goes out on the control stream, which no polling kernel can hold up; until a wait
        // confirms it, kernels poll for this object's chunks
        o->async_counter = true;
        if (after != before || first) {
            rc = publish_counter(c, *o, after, c->ctl_stream);
            if (rc != HPL_OK) return rc;
            c->ctl_unconfirmed = true;
        }
    } else {
        if (after != before || first) {
            rc = publish_counter(c, *o, after, c->stream);
            if (rc != HPL_OK) return rc;
        }
        o->landed = after;
    }
    return after_event(c);
}

int hpl_put_host(hpl_ctx* c, int64_t id, const void* buf, uint64_t bytes) {
    Object* o = nullptr;
    int rc = put_checks(c, id, buf, bytes, &o);
    if (rc != HPL_OK) return rc;
    if (!c->device) return HPL_ERR_CUDA;
    if (c->world > 1) return HPL_ERR_INVALID;   // host objects are copied into THIS rank's store: not in worker-per-GPU mode
    const bool first = !o->arrived;
    if (!first && !o->from_host) return HPL_ERR_INVALID;
    if (first) {
        o->ptr = arena_alloc(c, o->bytes);
        if (!o->ptr) return HPL_ERR_NOMEM;
        o->lib_owned = true;
        o->from_host = true;
        o->async_counter = true;
        rc = alloc_row(c, *o);
        if (rc != HPL_OK) {
            arena_release(c, o->ptr);
            o->ptr = nullptr;
            o->lib_owned = false;
            return rc;
        }
        // the row must be in the directory (with a zero counter) before any copy-stream counter update
        rc = flush_directory(c);
        if (rc != HPL_OK) return rc;
        CUDA_TRY(cudaEventRecord(c->copy_ev, c->ctl_stream));
        CUDA_TRY(cudaStreamWaitEvent(c->copy_stream, c->copy_ev, 0));
    }
    const uint64_t old_bytes = o->ready_bytes;
    const uint64_t chunk = c->cfg.chunk_bytes;
    // copy [old_bytes, bytes) in pieces that end on chunk boundaries and publish the chunks of each piece as
    // it lands.  A piece is several chunks (about 8 MiB): every counter update is a copy of its own on the copy
    // engine (~2.5 us), which at one per 2 MiB chunk would cost a fifth of the PCIe rate.
    const uint64_t piece = std::max<uint64_t>(chunk, ((8ull << 20) + chunk - 1) / chunk * chunk);
    uint64_t off = old_bytes;
    while (off < bytes) {
        uint64_t end = std::min<uint64_t>((off / piece + 1) * piece, bytes);
        CUDA_TRY(cudaMemcpyAsync((uint8_t*)o->ptr + off, (const uint8_t*)buf + off, end - off, cudaMemcpyHostToDevice, c->copy_stream));
        c->stats.h2d_bytes += end - off;
        const uint32_t done = end >= o->bytes ? o->C : (uint32_t)(end / chunk);
        const uint32_t before_piece = off >= o->bytes ? o->C : (uint32_t)(off / chunk);
        if (done != before_piece) {
            rc = publish_counter(c, *o, done, c->copy_stream);
            if (rc != HPL_OK) return rc;
        }
        off = end;
    }
    c->copy_pending = true;
    do_put_common(c, *o, bytes, first);
    return after_event(c);
}

int hpl_reduce(hpl_ctx* c, int64_t target, const int64_t* src_ids, int32_t n, int32_t k, int32_t op, int32_t dtype) {
    if (!c || !src_ids || n < 1 || k < 1 || k > n || target < 0) return HPL_ERR_INVALID;
    if (op < HPL_SUM || op > HPL_MAX || (dtype != HPL_F32 && dtype != HPL_BF16)) return HPL_ERR_INVALID;
    if (c->objects.count(target)) return HPL_ERR_EXISTS;
    std::vector<int64_t> srcs(src_ids, src_ids + n);
    {
        std::vector<int64_t> u = srcs;
        std::sort(u.begin(), u.end());
        if (std::adjacent_find(u.begin(), u.end()) != u.end()) return HPL_ERR_INVALID;
    }
    uint64_t bytes = 0;
    int live = 0;
    struct Src { int64_t t_arrival; int index; int64_t id; bool alive, arrived; uint32_t C; Object* o; };
    std::vector<Src> info;   // what the steps below need of each source, looked up once (entries of the object table do not move)
    info.reserve(n);
    for (int i = 0; i < n; ++i) {
        Object* o = find(c, srcs[i]);
        if (!o) return HPL_ERR_NOT_FOUND;
        if (o->dtype != dtype || (bytes && o->bytes != bytes) || o->kind == OBJ_RECEIVER) return HPL_ERR_INVALID;
        bytes = o->bytes;
        if (o->alive) ++live;
        info.push_back({o->t_arrival, i, o->id, o->alive, o->arrived, o->C, o});
    }
    if (live < 1) return HPL_ERR_INSUFFICIENT;
    const uint64_t elems = bytes / elem_size(dtype);

    Object t;
    t.id = target;
    t.worker = -1;
    t.bytes = elems * 4;
    t.dtype = HPL_F32;
    t.C = (uint32_t)((t.bytes + c->cfg.chunk_bytes - 1) / c->cfg.chunk_bytes);
    t.kind = OBJ_TARGET;
    t.lib_owned = true;
    t.arrived = true;   // the output is published at once, as a partial object (Section 3.4.2)
    t.t_arrival = (int64_t)c->now;
    t.ready_bytes = 0;
    t.seq = c->seq++;
    {
        t.home = c->world > 1 ? (int)(target % c->world) : 0;
        if (c->world > 1 && !c->rank_alive[t.home]) return HPL_ERR_FAILED_WORKER;
        t.ptr = arena_alloc(c, t.bytes, t.home);
        if (!t.ptr) return HPL_ERR_NOMEM;
        int rc = alloc_row(c, t);
        if (rc != HPL_OK) {
            arena_release(c, t.ptr);
            return rc;
        }
    }
    c->objects.emplace(target, t);

    ReduceOp r;
    r.target = target;
    int degree = c->cfg.reduce_degree;
    if (degree == 0)   // Section 4: picked per Reduce from the latency / bandwidth model and the object size
        degree = choose_reduce_degree(k, (double)bytes, (double)c->cfg.model_latency_ns * 1e-9, (double)c->cfg.model_bandwidth_bps);
    if (std::min<int64_t>(degree, k - 1) + 2 > (int64_t)kMaxStepsPerWave) {   // one node's operands must fit one task
        if (t.ptr) arena_release(c, t.ptr);
        if (t.row >= 0) c->free_rows.push_back(t.row);
        c->objects.erase(target);
        return HPL_ERR_INVALID;
    }
    r.sched.reset(new ReduceTreeSchedule(srcs, k, degree));
    r.red_op = op;
    r.in_dtype = dtype;
    r.elems = elems;
    r.C = info[0].C;                    // chunks of this Reduce follow its inputs (chunk_bytes of the input dtype)
    r.chunk_elems = (uint32_t)(std::min<uint64_t>(c->cfg.chunk_bytes, bytes) / elem_size(dtype));
    if (r.chunk_elems == 0) r.chunk_elems = 1;
    r.seq = c->seq++;
    ReduceOp* rp = &r;
    auto dl = [c, rp](int64_t o) { return logical_delivered_in(c, o, *rp); };
    for (const Src& x : info)
        if (!x.alive) r.sched->fail(x.id, 0, dl);  // sources lost before the call never take part
    std::vector<std::pair<std::pair<int64_t, int>, int64_t>> arrived;
    arrived.reserve(n);
    for (const Src& x : info)
        if (x.alive && x.arrived) arrived.push_back({{x.t_arrival, x.index}, x.id});
    std::sort(arrived.begin(), arrived.end());
    for (auto& a : arrived) r.sched->arrive(a.second);
    r.merged.assign(r.sched->k(), IntervalMap());
    r.partial_key.assign(r.sched->k(), 0);
    const uint64_t key = r.seq;
    for (const Src& x : info) x.o->consumers.push_back(key);
    c->reduce_of_target[target] = key;
    c->reduces.emplace(key, std::move(r));
    refresh_composed(c);
    return after_event(c);
}

int hpl_broadcast(hpl_ctx* c, int64_t src_id, const int64_t* dst_ids, int32_t n) {
    if (!c || !dst_ids || n < 1) return HPL_ERR_INVALID;
    Object* src = find(c, src_id);
    if (!src) return HPL_ERR_NOT_FOUND;
    if (c->bcast_of_src.count(src_id)) return HPL_ERR_EXISTS;
    for (int i = 0; i < n; ++i) {
        Object* d = find(c, dst_ids[i]);
        if (!d) return HPL_ERR_NOT_FOUND;
        if (d->bytes != src->bytes || d->dtype != src->dtype || d->kind != OBJ_PLAIN || d->arrived) return HPL_ERR_INVALID;
        for (int j = 0; j < i; ++j)
            if (dst_ids[j] == dst_ids[i]) return HPL_ERR_INVALID;
    }
    if (!src->alive) return HPL_ERR_FAILED_WORKER;
    BcastOp b;
    b.src = src_id;
    b.sched.reset(new BroadcastTreeSchedule(src_id, src->C, c->cfg.bcast_degree, (int64_t)c->tau));
    b.sched->advance((int64_t)c->now);
    if (src->arrived) b.sched->source_progress((int64_t)c->now, logical_delivered(c, src_id));
    b.dsts.assign(dst_ids, dst_ids + n);
    b.seq = c->seq++;
    for (int i = 0; i < n; ++i) {
        Object* d = find(c, dst_ids[i]);
        d->kind = OBJ_RECEIVER;
        d->op_key = src_id;
    }
    c->bcast_of_src[src_id] = b.seq;
    const uint64_t key = b.seq;
    if (src->kind == OBJ_TARGET) c->composed_bcasts.insert(key);   // an object's kind never changes while it is a source
    c->bcasts.emplace(key, std::move(b));
    return after_event(c);
}

int hpl_join(hpl_ctx* c, int64_t dst_id, void* dst_buf) {
    if (!c) return HPL_ERR_INVALID;
    Object* d = find(c, dst_id);
    if (!d) return HPL_ERR_NOT_FOUND;
    if (d->kind != OBJ_RECEIVER) return HPL_ERR_NOT_FOUND;
    if (!d->alive) return HPL_ERR_FAILED_WORKER;
    if (c->device && (!dst_buf || (uintptr_t)dst_buf % 16)) return HPL_ERR_INVALID;
    BcastOp& b = c->bcasts.at(c->bcast_of_src.at(d->op_key));
    const int li = b.sched->index_of(dst_id);
    if (li < 0 || !b.sched->locations()[li].alive) {   // first join, or again after its worker was rebuilt
        d->ptr = dst_buf;
        d->home = c->world > 1 ? d->worker % c->world : 0;
        d->ready_bytes = 0;
        int rc = alloc_row(c, *d);
        if (rc != HPL_OK) return rc;
    }
    b.sched->join((int64_t)c->now, dst_id);
    return after_event(c);
}

int hpl_fail(hpl_ctx* c, int32_t worker) {
    if (!c || worker < 0) return HPL_ERR_INVALID;
    if (!c->levels.empty()) return HPL_ERR_INVALID;   // worker-per-GPU mode: trees change between plans, not inside one
    std::vector<Object*> lost;
    for (auto& kv : c->objects)
        if (kv.second.worker == worker && kv.second.alive) lost.push_back(&kv.second);
    std::sort(lost.begin(), lost.end(), [](Object* a, Object* b) { return a->seq < b->seq; });
    if (c->world <= 1 && !lost.empty()) {
        // Copies are made lazily (at a Get, or at every event when eager), while in the schedule a receiver may already
        // hold chunks it was sent before this instant.  What a copy that is about to disappear can still serve is
        // therefore copied NOW, by work enqueued before the call returns: afterwards its buffer is never read again.
        bool any = false;
        for (auto& kv : c->bcasts) {
            BcastOp& op = kv.second;
            bool concerned = false;
            for (Object* o : lost) concerned = concerned || o->id == op.src || (o->kind == OBJ_RECEIVER && o->op_key == op.src);
            if (!concerned) continue;
            if (!any) {
                ++c->plan_pass;
                int rc = flush_directory(c);
                if (rc != HPL_OK) return rc;
                if (c->device && c->copy_pending && !c->cfg.plan_ahead) {
                    CUDA_TRY(cudaEventRecord(c->copy_ev, c->copy_stream));
                    CUDA_TRY(cudaStreamWaitEvent(c->stream, c->copy_ev, 0));
                    c->copy_pending = false;
                    for (auto& ob : c->objects)
                        if (ob.second.async_counter) ob.second.landed = published_chunks(c, ob.second);
                }
                any = true;
            }
            c->batch_tag = ++c->tag_counter;
            std::vector<PlannedFanout> tasks;
            int rc = plan_bcast(c, op, tasks);
            if (rc != HPL_OK) return rc;
            rc = launch_fanout_tasks(c, op, tasks);
            if (rc != HPL_OK) return rc;
        }
    }
    for (Object* o : lost) o->alive = false;
    for (auto& kv : c->reduces) {
        ReduceOp& op = kv.second;
        ReduceOp* rp = &op;
        auto dl = [c, rp](int64_t o) { return logical_delivered_in(c, o, *rp); };
        for (Object* o : lost) {
            if (!op.sched->has_source(o->id)) continue;
            ReduceInvalidation inv = op.sched->fail(o->id, logical_delivered_in(c, o->id, op), dl);
            apply_invalidation(c, op, inv);
            if (!inv.positions.empty() || inv.shrank) invalidate_consumers(c, op.target);
        }
    }
    for (auto& kv : c->bcasts) {
        BcastOp& op = kv.second;
        std::vector<int64_t> mine;
        for (Object* o : lost)
            if (o->id == op.src || (o->kind == OBJ_RECEIVER && o->op_key == op.src)) mine.push_back(o->id);
        if (!mine.empty()) op.sched->fail((int64_t)c->now, mine);
    }
    refresh_composed(c);
    return after_event(c);
}

int hpl_rejoin(hpl_ctx* c, int32_t worker) {
    if (!c || worker < 0) return HPL_ERR_INVALID;
    if (!c->levels.empty()) return HPL_ERR_INVALID;
    bool any = false;
    for (auto& kv : c->objects) {
        Object& o = kv.second;
        if (o.worker == worker && !o.alive && !c->bcast_of_src.count(o.id)) any = true;
    }
    if (!any) return HPL_OK;
    if (c->device) {   // rows and store copies of the revived objects are recycled: nothing may still read them
        cudaStreamSynchronize(c->ctl_stream);
        cudaStreamSynchronize(c->copy_stream);
        cudaStreamSynchronize(c->stream);
    }
    for (auto& kv : c->objects) {
        Object& o = kv.second;
        if (o.worker != worker || o.alive || c->bcast_of_src.count(o.id)) continue;
        release_object_memory(c, o);
        o.alive = true;
        o.arrived = false;
        o.ready_bytes = 0;
        o.landed = 0;
        o.t_arrival = -1;
        o.lib_owned = false;
        o.from_host = false;
        o.async_counter = false;
        const int64_t id = o.id;
        o.consumers.for_each([c, id](uint64_t key) {
            auto r = c->reduces.find(key);
            if (r != c->reduces.end()) r->second.sched->rejoin(id);
        });
    }
    return after_event(c);
}

int32_t hpl_choose_degree(int32_t n, uint64_t object_bytes, double latency_s, double bandwidth_bytes_per_s) {
    if (n < 1 || !(latency_s >= 0.0) || !(bandwidth_bytes_per_s > 0.0)) return HPL_ERR_INVALID;
    return choose_reduce_degree(n, (double)object_bytes, latency_s, bandwidth_bytes_per_s);
}

int hpl_create_batch(hpl_ctx* c, int32_t n, const int64_t* ids, const int32_t* workers, uint64_t total_bytes, int32_t dtype,
                     int32_t* n_done) {
    if (!c || n < 0 || (n && (!ids || !workers))) return HPL_ERR_INVALID;
    int rc = HPL_OK, i = 0;
    for (; i < n && rc == HPL_OK; ++i) rc = hpl_create(c, ids[i], workers[i], total_bytes, dtype);
    if (n_done) *n_done = rc == HPL_OK ? i : i - 1;
    return rc;
}

int hpl_put_batch(hpl_ctx* c, int32_t n, const int64_t* ids, const void* const* bufs, const uint64_t* bytes, int32_t* n_done) {
    if (!c || n < 0 || (n && (!ids || !bufs || !bytes))) return HPL_ERR_INVALID;
    int rc = HPL_OK, i = 0;
    for (; i < n && rc == HPL_OK; ++i) rc = hpl_put(c, ids[i], bufs[i], bytes[i]);
    if (n_done) *n_done = rc == HPL_OK ? i : i - 1;
    return rc;
}

int hpl_join_batch(hpl_ctx* c, int32_t n, const int64_t* ids, void* const* bufs, int32_t* n_done) {
    if (!c || n < 0 || (n && (!ids || !bufs))) return HPL_ERR_INVALID;
    int rc = HPL_OK, i = 0;
    for (; i < n && rc == HPL_OK; ++i) rc = hpl_join(c, ids[i], bufs[i]);
    if (n_done) *n_done = rc == HPL_OK ? i : i - 1;
    return rc;
}

int hpl_progress(hpl_ctx* c) {
    if (!c) return HPL_ERR_INVALID;
    return progress(c);
}

int hpl_sync(hpl_ctx* c) {
    if (!c) return HPL_ERR_INVALID;
    return sync_and_check(c);
}

int hpl_get(hpl_ctx* c, int64_t id, const void** dev_ptr, uint64_t* bytes) {
    if (!c) return HPL_ERR_INVALID;
    Object* o = find(c, id);
    if (!o) return HPL_ERR_NOT_FOUND;
    if (o->kind == OBJ_TARGET) {
        ReduceOp& op = c->reduces.at(c->reduce_of_target.at(id));
        if (op.sched->k() == 0) return HPL_ERR_INSUFFICIENT;
        if (c->device && !c->work_in_flight && !c->copy_pending && !c->ctl_unconfirmed && op.sched->full() &&
            op.merged[0].covers(0, op.C, op.n_ops(0))) {
            if (dev_ptr) *dev_ptr = o->ptr;   // computed and waited for already (e.g. by an earlier Get of a batch)
            if (bytes) *bytes = o->bytes;
            return HPL_OK;
        }
        if (op.lost) return HPL_ERR_FAILED_WORKER;
        int rc = c->world > 1 ? HPL_OK : progress(c);   // whatever can run now runs, even if the target cannot complete yet
        if (rc != HPL_OK) return rc;
        if (c->world > 1 && !c->levels.empty()) return HPL_ERR_TIMEOUT;   // the caller drives the levels (hpl_run_level)
        if (!op.sched->full()) return HPL_ERR_TIMEOUT;
        for (int p = 0; p < op.sched->k(); ++p) {
            Object* m = find(c, op.sched->object_at(p));
            if (!m || logical_ready_elems(c, m->id) < object_elems(*m)) return HPL_ERR_TIMEOUT;
        }
        if (!c->device) return HPL_ERR_CUDA;
        if (!op.merged[0].covers(0, op.C, op.n_ops(0))) return HPL_ERR_TIMEOUT;
        rc = sync_and_check(c);
        // a wait that expired in some other collective's wave does not concern this target if its own work stands
        if (rc == HPL_ERR_TIMEOUT && op.merged[0].covers(0, op.C, op.n_ops(0))) rc = HPL_OK;
        if (rc != HPL_OK) return rc;
    } else if (o->kind == OBJ_RECEIVER) {
        if (!o->alive) return HPL_ERR_FAILED_WORKER;
        BcastOp& op = c->bcasts.at(c->bcast_of_src.at(o->op_key));
        const int li = op.sched->index_of(id);
        // never asked, or its worker was rebuilt and has not asked again (a rebuilt receiver holds no copy until it joins
        // again as a new location, Section 3.5.1)
        if (li < 0 || !op.sched->locations()[li].alive) return HPL_ERR_TIMEOUT;
        if (c->world <= 1 && (li >= (int)op.phys_have.size() || op.phys_have[li] < (int64_t)o->C)) {
            // start the copies first: the GPU works while the host lets the virtual clock run below
            int rc = progress(c);
            if (rc != HPL_OK) return rc;
        }
        if (!op.sched->run_until_complete(id)) return HPL_ERR_TIMEOUT;
        if ((uint64_t)op.sched->now() > c->now) c->now = (uint64_t)op.sched->now();
        for (auto& kv : c->bcasts) kv.second.sched->advance((int64_t)c->now);
        {
            // a copy of a Reduce output is only complete while that output is (a member may have been lost since)
            Object* so = find(c, op.src);
            if (so && so->kind == OBJ_TARGET) {
                ReduceOp& up = c->reduces.at(c->reduce_of_target.at(op.src));
                if (up.sched->k() == 0) return HPL_ERR_INSUFFICIENT;
                if (logical_delivered(c, op.src) < (int64_t)so->C) return HPL_ERR_TIMEOUT;
            }
        }
        if (c->world > 1 && (!c->levels.empty() || li >= (int)op.phys_have.size() || op.phys_have[li] < (int64_t)o->C))
            return HPL_ERR_TIMEOUT;   // worker-per-GPU mode: the caller drives the levels (hpl_run_level)
        if (!c->device) return HPL_ERR_CUDA;
        if (li < (int)op.phys_have.size() && op.phys_have[li] >= (int64_t)o->C && !c->work_in_flight && !c->copy_pending) {
            if (dev_ptr) *dev_ptr = o->ptr;   // already copied and waited for
            if (bytes) *bytes = o->bytes;
            return HPL_OK;
        }
        int rc = c->world > 1 ? HPL_OK : progress(c);
        if (rc != HPL_OK) return rc;
        if (li >= (int)op.phys_have.size() || op.phys_have[li] < (int64_t)o->C) return HPL_ERR_TIMEOUT;
        rc = sync_and_check(c);
        if (rc == HPL_ERR_TIMEOUT && op.phys_have[li] >= (int64_t)o->C) rc = HPL_OK;   // the expired wait was elsewhere
        if (rc != HPL_OK) return rc;
    } else {
        if (!o->alive) return HPL_ERR_FAILED_WORKER;
        if (!o->arrived || o->ready_bytes < o->bytes) return HPL_ERR_TIMEOUT;
        if (!c->device) return HPL_ERR_CUDA;
        int rc = sync_and_check(c);
        if (rc != HPL_OK) return rc;
    }
    if (dev_ptr) *dev_ptr = o->ptr;
    if (bytes) *bytes = o->bytes;
    return HPL_OK;
}

int hpl_get_batch(hpl_ctx* c, int32_t n, const int64_t* ids, const void** dev_ptrs, int32_t* n_done) {
    if (!c || n < 0 || (n && !ids)) return HPL_ERR_INVALID;
    int rc = HPL_OK, i = 0;
    for (; i < n && rc == HPL_OK; ++i) rc = hpl_get(c, ids[i], dev_ptrs ? &dev_ptrs[i] : nullptr, nullptr);
    if (n_done) *n_done = rc == HPL_OK ? i : i - 1;
    return rc;
}

int hpl_submit(hpl_ctx* c, hpl_event* ev, int32_t n, int32_t* n_done) {
    if (!c || n < 0 || (n && !ev)) return HPL_ERR_INVALID;
    int rc = HPL_OK, done = 0;
    for (int i = 0; i < n; ++i) {
        hpl_event& e = ev[i];
        if (e.t_ns != 0 && e.t_ns != c->now) {
            rc = hpl_advance(c, e.t_ns);
            if (rc != HPL_OK) break;
        }
        switch (e.kind) {
            case HPL_EV_CREATE: rc = hpl_create(c, e.object_id, e.worker, e.bytes, e.dtype); break;
            case HPL_EV_PUT: rc = hpl_put(c, e.object_id, e.ptr, e.bytes); break;
            case HPL_EV_PUT_HOST: rc = hpl_put_host(c, e.object_id, e.ptr, e.bytes); break;
            case HPL_EV_REDUCE: rc = hpl_reduce(c, e.object_id, e.ids, e.n_ids, e.k, e.op, e.dtype); break;
            case HPL_EV_BROADCAST: rc = hpl_broadcast(c, e.object_id, e.ids, e.n_ids); break;
            case HPL_EV_JOIN: rc = hpl_join(c, e.object_id, e.ptr); break;
            case HPL_EV_FAIL: rc = hpl_fail(c, e.worker); break;
            case HPL_EV_REJOIN: rc = hpl_rejoin(c, e.worker); break;
            case HPL_EV_PROGRESS: rc = hpl_progress(c); break;
            case HPL_EV_GET: {
                const void* p = nullptr;
                uint64_t nb = 0;
                rc = hpl_get(c, e.object_id, &p, &nb);
                if (rc == HPL_OK) {
                    e.ptr = const_cast<void*>(p);
                    e.bytes = nb;
                }
                break;
            }
            case HPL_EV_DELETE: rc = hpl_delete(c, e.object_id); break;
            case HPL_EV_SYNC: rc = hpl_sync(c); break;
            case HPL_EV_MARK:
                if (c->device && (!e.ptr || cudaEventRecord((cudaEvent_t)e.ptr, c->stream) != cudaSuccess)) rc = HPL_ERR_CUDA;
                break;
            default: rc = HPL_ERR_INVALID;
        }
        if (rc != HPL_OK) break;
        ++done;
    }
    if (n_done) *n_done = done;
    return rc;
}

int hpl_get_host(hpl_ctx* c, int64_t id, void* dst, uint64_t cap) {
    if (!c || !dst) return HPL_ERR_INVALID;
    const void* p = nullptr;
    uint64_t n = 0;
    int rc = hpl_get(c, id, &p, &n);
    if (rc != HPL_OK) return rc;
    if (cap < n) return HPL_ERR_INVALID;
    CUDA_TRY(cudaMemcpyAsync(dst, p, n, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    c->stats.d2h_bytes += n;
    return HPL_OK;
}

int hpl_delete(hpl_ctx* c, int64_t id) {
    if (!c) return HPL_ERR_INVALID;
    Object* o = find(c, id);
    if (!o || id < 0) return HPL_ERR_NOT_FOUND;
    if (!c->levels.empty()) return HPL_ERR_INVALID;       // worker-per-GPU mode: a planned level may still name it
    if (o->kind == OBJ_RECEIVER) return HPL_ERR_INVALID;  // deleted with its broadcast
    if (!o->consumers.empty()) return HPL_ERR_INVALID;  // still referenced by a Reduce
    if (c->device && (c->work_in_flight || c->copy_pending || c->ctl_unconfirmed)) {
        // rows and arena memory are recycled only when nothing enqueued can still read them (nothing of the
        // library's is in flight after a Get or a wait, so a round's Deletes cost no device wait)
        cudaStreamSynchronize(c->ctl_stream);
        cudaStreamSynchronize(c->copy_stream);
        cudaStreamSynchronize(c->stream);
    }
    if (o->kind == OBJ_TARGET) {
        const uint64_t key = c->reduce_of_target.at(id);
        ReduceOp& op = c->reduces.at(key);
        for (int64_t pk : op.partial_key)
            if (pk != 0) {
                Object* po = find(c, pk);
                if (po) {
                    release_object_memory(c, *po);
                    c->objects.erase(pk);
                }
            }
        for (int64_t sid : op.sched->sources()) {
            Object* so = find(c, sid);
            if (so) so->consumers.erase(key);
        }
        c->reduces.erase(key);
        c->reduce_of_target.erase(id);
    }
    auto b = c->bcast_of_src.find(id);
    if (b != c->bcast_of_src.end()) {
        BcastOp& op = c->bcasts.at(b->second);
        for (int64_t d : op.dsts) {
            Object* r = find(c, d);
            if (r) {
                release_object_memory(c, *r);
                c->objects.erase(d);
            }
        }
        c->composed_bcasts.erase(b->second);
        c->bcasts.erase(b->second);
        c->bcast_of_src.erase(b);
    }
    o = find(c, id);
    release_object_memory(c, *o);
    c->objects.erase(id);
    return HPL_OK;
}

int hpl_schedule_dump(hpl_ctx* c, int64_t op_id, int64_t* words, uint64_t cap, uint64_t* len) {
    if (!c || !len) return HPL_ERR_INVALID;
    std::vector<int64_t> w;
    auto r = c->reduce_of_target.find(op_id);
    auto b = c->bcast_of_src.find(op_id);
    if (r != c->reduce_of_target.end())
        c->reduces.at(r->second).sched->dump(op_id, w);
    else if (b != c->bcast_of_src.end())
        c->bcasts.at(b->second).sched->dump(w);
    else {
        // a receiver names the broadcast it belongs to (the only handle on it when the source is a Reduce output)
        Object* o = find(c, op_id);
        if (!o || o->kind != OBJ_RECEIVER) return HPL_ERR_NOT_FOUND;
        auto bo = c->bcast_of_src.find(o->op_key);
        if (bo == c->bcast_of_src.end()) return HPL_ERR_NOT_FOUND;
        c->bcasts.at(bo->second).sched->dump(w);
    }
    *len = w.size();
    if (!words || cap < w.size()) return HPL_ERR_INVALID;
    std::memcpy(words, w.data(), w.size() * sizeof(int64_t));
    return HPL_OK;
}

int hpl_set_peer_arena(hpl_ctx* c, int32_t rank, void* base) {
    if (!c || c->world <= 1 || rank < 0 || rank >= c->world || rank == c->rank || !base || (uintptr_t)base % kAlign) return HPL_ERR_INVALID;
    Arena& ar = c->peer_arenas[rank];
    if (ar.sizes_.size() != 2) return HPL_ERR_INVALID;   // addresses in it have been handed out already
    ar.base = (uint8_t*)base;
    return HPL_OK;
}

int hpl_pending_levels(hpl_ctx* c, int32_t* levels) {
    if (!c || !levels) return HPL_ERR_INVALID;
    *levels = (int32_t)c->levels.size();
    return HPL_OK;
}

int hpl_run_level(hpl_ctx* c) {
    if (!c || c->world <= 1) return HPL_ERR_INVALID;
    return run_level(c);
}

int hpl_fail_rank(hpl_ctx* c, int32_t rank) {
    if (!c || c->world <= 1 || rank < 0 || rank >= c->world) return HPL_ERR_INVALID;
    if (!c->levels.empty()) return HPL_ERR_INVALID;   // a rank leaves between plans, with no level pending
    if (!c->rank_alive[rank]) return HPL_OK;
    if (c->device) {
        cudaStreamSynchronize(c->ctl_stream);
        cudaStreamSynchronize(c->stream);
    }
    c->rank_alive[rank] = 0;
    // what the library itself kept on that GPU: outputs are lost with it, partial results are made again elsewhere
    for (auto& kv : c->reduces) {
        ReduceOp& op = kv.second;
        Object* tgt = find(c, op.target);
        if (tgt && tgt->home == rank) {
            op.lost = true;
            invalidate_consumers(c, op.target);
        }
        ReduceInvalidation inv;
        for (int p = 0; p < (int)op.partial_key.size(); ++p) {
            if (op.partial_key[p] == 0) continue;
            Object* po = find(c, op.partial_key[p]);
            if (!po || po->home != rank) continue;
            release_object_memory(c, *po);
            c->objects.erase(op.partial_key[p]);
            op.partial_key[p] = 0;
            inv.touched.push_back(p);
        }
        if (!inv.touched.empty()) {
            apply_invalidation(c, op, inv);
            invalidate_consumers(c, op.target);
        }
    }
    // its task workers fail (Section 3.5)
    std::vector<int32_t> workers;
    for (auto& kv : c->objects)
        if (kv.second.alive && kv.second.worker >= 0 && kv.second.worker % c->world == rank) workers.push_back(kv.second.worker);
    std::sort(workers.begin(), workers.end());
    workers.erase(std::unique(workers.begin(), workers.end()), workers.end());
    for (int32_t w : workers) {
        int rc = hpl_fail(c, w);
        if (rc != HPL_OK) return rc;
    }
    return HPL_OK;
}

int hpl_ipc_export(const void* dev_ptr, uint8_t handle[64], uint64_t* offset) {
    static_assert(sizeof(cudaIpcMemHandle_t) == 64, "IPC handle size");
    if (!dev_ptr || !handle || !offset) return HPL_ERR_INVALID;
    // the start of the allocation: asked of the driver, which is looked up at run time (the library itself links
    // the runtime only, so that it loads on a machine without a GPU)
    typedef int (*range_fn)(unsigned long long*, size_t*, unsigned long long);
    static range_fn get_range = nullptr;
    static std::once_flag looked_up;
    std::call_once(looked_up, [] {
        void* drv = dlopen("libcuda.so.1", RTLD_NOW | RTLD_GLOBAL);
        if (drv) get_range = (range_fn)dlsym(drv, "cuMemGetAddressRange_v2");
    });
    unsigned long long base = 0;
    size_t size = 0;
    if (!get_range || get_range(&base, &size, (unsigned long long)(uintptr_t)dev_ptr) != 0) return HPL_ERR_CUDA;
    cudaIpcMemHandle_t h;
    CUDA_TRY(cudaIpcGetMemHandle(&h, (void*)(uintptr_t)base));
    std::memcpy(handle, &h, 64);
    *offset = (uint64_t)((uintptr_t)dev_ptr - base);
    return HPL_OK;
}

namespace {
std::mutex g_ipc_mu;
std::map<void*, void*> g_ipc_base_of;   // address handed out by hpl_ipc_import -> start of the mapping
}

int hpl_ipc_import(const uint8_t handle[64], uint64_t offset, void** dev_ptr) {
    if (!handle || !dev_ptr) return HPL_ERR_INVALID;
    cudaIpcMemHandle_t h;
    std::memcpy(&h, handle, 64);
    void* base = nullptr;
    CUDA_TRY(cudaIpcOpenMemHandle(&base, h, cudaIpcMemLazyEnablePeerAccess));
    *dev_ptr = (uint8_t*)base + offset;
    std::lock_guard<std::mutex> lock(g_ipc_mu);
    g_ipc_base_of[*dev_ptr] = base;
    return HPL_OK;
}

int hpl_ipc_close(void* dev_ptr) {
    if (!dev_ptr) return HPL_ERR_INVALID;
    void* base = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_ipc_mu);
        auto it = g_ipc_base_of.find(dev_ptr);
        if (it == g_ipc_base_of.end()) return HPL_ERR_NOT_FOUND;
        base = it->second;
        g_ipc_base_of.erase(it);
    }
    CUDA_TRY(cudaIpcCloseMemHandle(base));
    return HPL_OK;
}

int hpl_check_guards(hpl_ctx* c, uint64_t* violations) {
    if (!c || !violations) return HPL_ERR_INVALID;
    if (c->device)
        for (auto& g : c->guards) c->guard_violations += check_guard(c, g.first);
    *violations = c->guard_violations;
    return HPL_OK;
}

int hpl_stats(hpl_ctx* c, hpl_stats_t* out) {
    if (!c || !out) return HPL_ERR_INVALID;
    c->stats.arena_used = c->arena.used;
    *out = c->stats;
    return HPL_OK;
}

}  // extern "C"
