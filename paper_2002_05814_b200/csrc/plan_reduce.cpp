// Reduce planner: turns the current state of a reduce tree into waves of fused subtree tasks.
#include "context.h"

namespace hpl {

struct ReducePlanCtx {
    hpl_ctx* c;
    ReduceOp* op;
    uint32_t a, b;                 // chunk interval being planned
    std::vector<uint32_t> ready;   // per position: chunks that may be consumed
    std::vector<uint32_t> landed;  // per position: chunks known to be visible without polling
    std::vector<int> m0;           // per position: operands already merged into its buffer over [a, b)
    std::vector<int> prefix;       // per position: operands that could be merged now (>= m0)
    std::vector<char> full, avail; // result complete already / could be completed now
    std::vector<int> level_of;     // level at which the position's complete result becomes available in this pass
    std::vector<PlannedReduceTask>* out;
    int err = HPL_OK;
};

int ensure_partial_buffer(hpl_ctx* c, ReduceOp& op, int pos, Object** out) {
    if (pos == 0) {
        *out = find(c, op.target);
        return HPL_OK;
    }
    if (op.partial_key[pos] != 0) {
        *out = find(c, op.partial_key[pos]);
        (*out)->last_use = ++c->use_tick;
        (*out)->last_pass = c->plan_pass;
        return HPL_OK;
    }
    Object o;
    o.id = c->next_internal--;
    o.kind = OBJ_PARTIAL;
    o.op_key = op.target;
    o.pos = pos;
    o.last_use = ++c->use_tick;
    o.last_pass = c->plan_pass;
    o.bytes = op.elems * 4;
    o.dtype = HPL_F32;
    o.C = op.C;
    o.lib_owned = true;
    o.seq = c->seq++;
    if (c->world > 1) {   // the partial result of a tree node lives with the node's object (else with the output)
        Object* own = find(c, op.sched->object_at(pos));
        Object* tgt = find(c, op.target);
        o.home = own ? own->home : (tgt ? tgt->home : c->rank);
        if (!c->rank_alive[o.home] && tgt) o.home = tgt->home;
    }
    o.ptr = arena_alloc(c, o.bytes, c->world > 1 ? o.home : -1);
    if (!o.ptr) return HPL_ERR_NOMEM;
    o.ready_bytes = o.bytes;
    int rc = alloc_row(c, o);
    if (rc != HPL_OK) {
        arena_release(c, o.ptr);
        return rc;
    }
    op.partial_key[pos] = o.id;
    auto ins = c->objects.emplace(o.id, o);
    *out = &ins.first->second;
    return HPL_OK;
}

int ensure_result(ReducePlanCtx& p, int v, int end);

// One load step: the position's own object (partial == false) or the buffer that holds its (partial) result.
void emit_operand(ReducePlanCtx& p, PlannedReduceTask& task, int q, bool partial, uint8_t code, int acc) {
    ReduceOp& op = *p.op;
    ReduceStep st{};
    st.code = code;
    st.a = (uint8_t)acc;
    if (partial) {
        st.kind = SRC_F32;
        Object* o = find(p.c, q == 0 ? op.target : op.partial_key[q]);
        o->last_use = ++p.c->use_tick;
        o->last_pass = p.c->plan_pass;
        st.row = (uint32_t)o->row;
        st.ptr = (unsigned long long)(uintptr_t)o->ptr;
    } else {
        st.kind = op.in_dtype == HPL_BF16 ? SRC_BF16 : SRC_F32;
        const Object* o = find(p.c, op.sched->object_at(q));
        st.row = (uint32_t)o->row;
        st.ptr = (unsigned long long)(uintptr_t)o->ptr;
        if (p.landed[q] < p.b) task.poll = true;  // not yet known to be visible: the kernel polls its counter
    }
    task.steps.push_back(st);
}

// Nodes in the subtree of position q of the complete d-ary tree on k positions.
int64_t subtree_size(const ReduceTreeSchedule& s, int q) {
    int64_t total = 0, lo = q, hi = q;
    const int64_t k = s.k(), d = s.d();
    while (lo < k) {
        total += std::min(hi, k - 1) - lo + 1;
        lo = d * lo + 1;
        hi = d * hi + d;
    }
    return total;
}

// Emits the steps that merge operands [m0[u], end) of node u into accumulator `acc`, starting from the buffer
// of u when some operands are merged already.  `budget`: steps this subtree may still add (a task must fit one
// wave's step table).  A child subtree that cannot be fused (fusion off, no accumulator left, no room) is
// completed by a task of its own first.
void gen_steps(ReducePlanCtx& p, int u, int acc, int end, PlannedReduceTask& task, int& dep_level, int64_t budget) {
    ReduceTreeSchedule& s = *p.op->sched;
    auto is_complete = [&](int q) { return !s.is_leaf(q) && (p.full[q] || p.level_of[q] >= 0); };
    const int64_t begin = (int64_t)task.steps.size();
    task.n_acc = std::max(task.n_acc, acc + 1);
    if (s.is_leaf(u)) {
        emit_operand(p, task, u, false, OPC_LOAD, acc);
        return;
    }
    bool first = true;
    if (p.m0[u] > 0) {   // continue from what the node's buffer already holds
        emit_operand(p, task, u, true, OPC_LOAD, acc);
        first = false;
    }
    for (int i = p.m0[u]; i < end; ++i) {
        const uint8_t code = first ? OPC_LOAD : OPC_ADD_LOAD;
        const int cj = operand_child(s, u, i);
        if (cj < 0) {
            emit_operand(p, task, u, false, code, acc);
        } else if (s.is_leaf(cj)) {
            emit_operand(p, task, cj, false, code, acc);
        } else {
            const int acc_j = first ? acc : acc + 1;   // where a fused subtree of this child would live
            const int64_t used = (int64_t)task.steps.size() - begin;
            const int64_t avail = budget - used - 2 * (int64_t)(end - 1 - i) - 1;
            const bool fits = 2 * subtree_size(s, cj) + 1 <= avail;
            if (!is_complete(cj) && (!p.c->cfg.fuse || acc_j >= kMaxAcc || !fits)) ensure_result(p, cj, p.op->n_ops(cj));
            if (p.err != HPL_OK) return;
            if (is_complete(cj)) {
                if (p.level_of[cj] > dep_level) dep_level = p.level_of[cj];
                emit_operand(p, task, cj, true, code, acc);
            } else {
                gen_steps(p, cj, acc_j, p.op->n_ops(cj), task, dep_level, avail);
                if (!first) {
                    ReduceStep st{};
                    st.code = OPC_ADD_ACC;
                    st.a = (uint8_t)acc;
                    st.b = (uint8_t)acc_j;
                    task.steps.push_back(st);
                }
            }
        }
        first = false;
    }
}

// Plans the task that merges operands up to `end` into the buffer of position v over [a, b); returns the level
// (>= 1) at which that buffer is ready.
int ensure_result(ReducePlanCtx& p, int v, int end) {
    if (p.err != HPL_OK) return 0;
    const bool complete = end == p.op->n_ops(v);
    if (p.full[v]) return 0;
    if (p.level_of[v] >= 0) return p.level_of[v];
    Object* outbuf = nullptr;
    int rc = ensure_partial_buffer(p.c, *p.op, v, &outbuf);
    if (rc != HPL_OK) {
        p.err = rc;
        return 0;
    }
    PlannedReduceTask task;
    task.pos = v;
    task.end = end;
    task.a = p.a;
    task.b = p.b;
    task.n_acc = 1;
    task.poll = false;
    int dep = 0;
    gen_steps(p, v, 0, end, task, dep, kMaxStepsPerWave);
    if (p.err == HPL_OK && task.steps.size() > (size_t)kMaxStepsPerWave) p.err = HPL_ERR_INVALID;   // a node with more children than a task holds
    task.level = dep + 1;
    if (complete) p.level_of[v] = task.level;
    p.out->push_back(std::move(task));
    return task.level;
}

// Whatever can run now: a node whose remaining operands are all available is completed (its whole ready
// subtree fused into one task); otherwise the operands that are available, in order, are merged into its
// buffer (each arriving part is reduced into the parent's partial result), and the search goes on below.
void visit_for_progress(ReducePlanCtx& p, int v) {
    ReduceTreeSchedule& s = *p.op->sched;
    if (s.is_leaf(v) || p.full[v]) return;
    if (p.avail[v]) {
        ensure_result(p, v, p.op->n_ops(v));
        return;
    }
    int merged = p.m0[v];
    if (p.prefix[v] > p.m0[v] && p.prefix[v] >= 2) {
        ensure_result(p, v, p.prefix[v]);
        merged = p.prefix[v];
    }
    const int nops = p.op->n_ops(v);
    for (int i = merged; i < nops; ++i) {
        const int cj = operand_child(s, v, i);
        if (cj >= 0) visit_for_progress(p, cj);
    }
}

// Reduce followed by broadcast (Section 3.4.3): receivers of a broadcast of this Reduce's output that need exactly
// the elements a root task is about to produce take them from that task -- its result tile goes to the target and
// to them in one pass, instead of being written and read again by a fan-out wave.  Returns the receivers' buffer
// addresses (at most `room`); their holdings are advanced like those of a planned fan-out task.
static void claim_fused_receivers(hpl_ctx* c, ReduceOp& op, PlannedReduceTask& t) {
    std::vector<unsigned long long>& out = t.fan;
    const size_t room = kMaxFusedDst;
    out.clear();
    t.fan_rows.clear();
    if (!c->cfg.fuse_fanout || t.pos != 0 || t.end != op.n_ops(0)) return;
    auto bi = c->bcast_of_src.find(op.target);
    if (bi == c->bcast_of_src.end()) return;
    BcastOp& b = c->bcasts.at(bi->second);
    Object* tgt = find(c, op.target);
    if (!tgt || !tgt->alive) return;
    // the task's elements in chunks of the broadcast (the output's own chunks)
    const uint64_t cbe = object_chunk_elems(c, *tgt);
    const uint64_t e_lo = (uint64_t)t.a * op.chunk_elems, e_hi = std::min<uint64_t>((uint64_t)t.b * op.chunk_elems, op.elems);
    if (e_lo % cbe != 0 || (e_hi % cbe != 0 && e_hi != op.elems)) return;
    const int64_t a_b = (int64_t)(e_lo / cbe), b_b = e_hi == op.elems ? (int64_t)tgt->C : (int64_t)(e_hi / cbe);
    const auto& locs = b.sched->locations();
    b.phys_have.resize(locs.size(), 0);
    for (size_t r = 1; r < locs.size() && out.size() < room; ++r) {
        if (!locs[r].alive || locs[r].last_sender < 0 || b.phys_have[r] != a_b) continue;
        Object* o = find(c, locs[r].obj);
        if (!o || !o->alive || !o->ptr || o->row < 0) continue;
        c->journal.b.push_back({b.src, (int)r, b.phys_have[r], c->batch_tag});
        b.phys_have[r] = b_b;
        out.push_back((unsigned long long)(uintptr_t)o->ptr);
        t.fan_rows.push_back((uint32_t)o->row);
    }
}

int plan_reduce(hpl_ctx* c, ReduceOp& op, std::vector<PlannedReduceTask>& tasks) {
    ReduceTreeSchedule& s = *op.sched;
    const int k = s.k();
    if (k <= 0 || op.lost) return HPL_OK;
    struct Planning {   // partial results of the Reduce being planned are not evicted under its feet
        hpl_ctx* c;
        Planning(hpl_ctx* ctx, int64_t t) : c(ctx) { c->planning_target = t; }
        ~Planning() { c->planning_target = -1; }
    } planning(c, op.target);
    // scratch that keeps its memory between calls (planning is not re-entrant: one pass at a time per thread)
    static thread_local std::vector<uint32_t> ready, landed, bp;
    static thread_local ReducePlanCtx p;
    ready.assign(k, 0);
    landed.assign(k, 0);
    bp.assign({0u, op.C});
    for (int p = 0; p < k; ++p) {
        op.merged[p].breakpoints(bp);
        const int64_t oid = s.object_at(p);
        if (oid < 0) continue;
        Object* o = find(c, oid);
        if (!o || !o->alive || !o->ptr || o->row < 0) continue;
        if (o->kind == OBJ_TARGET) {   // composed Reduce: the member is the output of an earlier Reduce
            const uint64_t n = produced_elems(c, *o);
            landed[p] = ready[p] = n >= op.elems ? op.C : (uint32_t)(n / op.chunk_elems);
        } else {
            const uint32_t pub = published_chunks(c, *o);
            landed[p] = std::min(pub, o->landed);
            ready[p] = c->cfg.plan_ahead ? o->C : landed[p];
        }
        bp.push_back(ready[p]);
        bp.push_back(landed[p]);
    }
    std::sort(bp.begin(), bp.end());
    bp.erase(std::unique(bp.begin(), bp.end()), bp.end());

    for (size_t i = 0; i + 1 < bp.size(); ++i) {
        p.err = HPL_OK;
        p.c = c;
        p.op = &op;
        p.a = bp[i];
        p.b = bp[i + 1];
        if (p.b > op.C) break;
        p.ready = ready;
        p.landed = landed;
        p.m0.assign(k, 0);
        p.prefix.assign(k, 0);
        p.full.assign(k, 0);
        p.avail.assign(k, 0);
        p.level_of.assign(k, -1);
        std::vector<PlannedReduceTask> local;
        p.out = &local;
        for (int q = k - 1; q >= 0; --q) {   // children have larger indices than their parent
            const int nops = op.n_ops(q);
            p.m0[q] = op.merged[q].value_at(p.a);
            p.full[q] = p.m0[q] == nops ? 1 : 0;
            if (s.is_leaf(q)) {
                p.avail[q] = ready[q] >= p.b ? 1 : 0;
                p.prefix[q] = p.avail[q] ? 1 : 0;
                continue;
            }
            int m1 = p.m0[q];
            while (m1 < nops) {
                const int cj = operand_child(s, q, m1);
                const bool ok = cj < 0 ? ready[q] >= p.b : (s.is_leaf(cj) ? ready[cj] >= p.b : (p.full[cj] || p.avail[cj]));
                if (!ok) break;
                ++m1;
            }
            p.prefix[q] = m1;
            p.avail[q] = m1 == nops ? 1 : 0;
        }
        if (s.is_leaf(0)) {
            // k == 1: the target is a copy of the only member
            if (!p.full[0] && p.avail[0]) ensure_result(p, 0, 1);
        } else {
            visit_for_progress(p, 0);
        }
        p.out = nullptr;   // (the scratch outlives this call; `local` does not)
        if (p.err != HPL_OK) return p.err;
        for (auto& t : local) {
            c->journal.r.push_back({op.target, t.pos, t.a, t.b, p.m0[t.pos], c->batch_tag});
            op.merged[t.pos].set(t.a, t.b, t.end);
            // merge with the previous interval's task for the same position when the program is the same
            bool merged = false;
            for (auto& prev : tasks) {
                if (prev.pos == t.pos && prev.end == t.end && prev.b == t.a && prev.level == t.level && prev.poll == t.poll &&
                    prev.steps.size() == t.steps.size() &&
                    std::memcmp(prev.steps.data(), t.steps.data(), t.steps.size() * sizeof(ReduceStep)) == 0) {
                    prev.b = t.b;
                    merged = true;
                    break;
                }
            }
            if (!merged) tasks.push_back(std::move(t));
        }
    }
    for (auto& t : tasks) claim_fused_receivers(c, op, t);   // on the final tasks: a claim is for exactly the task's elements
    return HPL_OK;
}

int occ_index(int n_acc) { return n_acc <= 2 ? 0 : (n_acc <= 4 ? 1 : 2); }

// Packs the tasks of one dependency level (of one collective, or of several small ones) into waves and launches
// them.  All tasks of a group read inputs of one dtype class (`bf16`); every task carries its own geometry.
int launch_reduce_group(hpl_ctx* c, std::vector<std::pair<ReduceOp*, PlannedReduceTask*>>& lv, bool bf16) {
    size_t i = 0;
    while (i < lv.size()) {
        static thread_local ReduceWave w;
        w.dir = c->d_dir;
        w.status = nullptr;
        w.budget_ns = c->cfg.poll_budget_ns;
        w.n_tasks = 0;
        w.total_tiles = 0;
        uint32_t n_steps = 0, n_fan = 0;
        int n_acc = 1;
        while (i < lv.size() && w.n_tasks < (uint32_t)kMaxTasksPerWave &&
               n_steps + lv[i].second->steps.size() <= (size_t)kMaxStepsPerWave && n_fan + lv[i].second->fan.size() <= (size_t)kMaxFusedDst) {
            ReduceOp& op = *lv[i].first;
            PlannedReduceTask& t = *lv[i].second;
            const uint32_t tpc_full = (op.chunk_elems + kTileElems - 1) / kTileElems;
            Object* out = nullptr;
            int rc = ensure_partial_buffer(c, op, t.pos, &out);
            if (rc != HPL_OK) return rc;
            ReduceTask& d = w.tasks[w.n_tasks++];
            d.out_ptr = (unsigned long long)(uintptr_t)out->ptr;
            d.elems = op.elems;
            d.chunk_elems = op.chunk_elems;
            d.c_begin = t.a;
            d.c_end = t.b;
            d.tiles_per_chunk = tpc_full;
            d.tile_begin = w.total_tiles;
            d.step_begin = n_steps;
            d.n_steps = (uint32_t)t.steps.size();
            d.red_op = (uint32_t)op.red_op;
            d.poll = t.poll ? 1u : 0u;
            if (t.poll) c->polling_in_flight = true;
            const std::vector<unsigned long long>& fan = t.fan;
            d.fan_begin = n_fan;
            d.n_fan = (uint32_t)fan.size();
            for (size_t q = 0; q < fan.size(); ++q) {
                w.fan_rows[n_fan] = t.fan_rows[q];
                w.fan_ptrs[n_fan++] = fan[q];
            }
            d.out_row = (uint32_t)out->row;
            for (size_t q = 0; q < t.steps.size(); ++q) {
                w.recs[n_steps + q] = pack_step(t.steps[q]);
                w.rows[n_steps + q] = t.steps[q].row;
            }
            n_steps += d.n_steps;
            w.total_tiles += (t.b - t.a) * tpc_full;
            n_acc = std::max(n_acc, t.n_acc);
            // accounting: bytes the task moves
            uint64_t e_lo = (uint64_t)t.a * op.chunk_elems, e_hi = std::min<uint64_t>((uint64_t)t.b * op.chunk_elems, op.elems);
            for (auto& st : t.steps)
                if (st.code != OPC_ADD_ACC) c->stats.bytes_read_planned += (e_hi - e_lo) * (st.kind == SRC_BF16 ? 2 : 4);
            c->stats.bytes_written_planned += (e_hi - e_lo) * 4 * (1 + fan.size());
            c->stats.reduce_tasks++;
            if (!fan.empty()) c->stats.fused_fanout_tasks++;
            ++i;
        }
        if (w.n_tasks == 0) return HPL_ERR_INVALID;  // a single task larger than a wave: tree too wide
        if (!c->device) {   // schedule-only context: the wave is planned and counted, not run
            c->stats.kernel_launches++;
            c->stats.reduce_launches++;
            c->stats.tiles += w.total_tiles;
            continue;
        }
        const bool fanned = n_fan != 0;
        int& occ = c->occ_reduce[bf16 ? 1 : 0][fanned ? 1 : 0][occ_index(n_acc)];
        if (occ == 0) occ = reduce_ctas_per_sm(n_acc, bf16, fanned);
        int grid = (int)std::min<uint64_t>(w.total_tiles, (uint64_t)c->n_sm * occ);
        if (grid < 1) grid = 1;
        if (flush_directory(c) != HPL_OK) return HPL_ERR_CUDA;   // rows of partial results created while planning
        bool polls = kDebugBounds;   // (the bounds-checking build reads the directory in every wave, and may record an error)
        for (uint32_t q = 0; q < w.n_tasks; ++q) polls = polls || w.tasks[q].poll;
        if (polls && order_main_after_control(c) != HPL_OK) return HPL_ERR_CUDA;   // the counters it waits on are rows of the directory
        if (kDebugBounds) c->polling_in_flight = true;
        w.status = next_wave_status(c);
        {
            LaunchTimer timer(c, 0);
            if (launch_reduce_wave(w, n_acc, bf16, fanned, grid, c->stream) != 0) return HPL_ERR_CUDA;
        }
        c->stats.kernel_launches++;
        c->stats.reduce_launches++;
        c->stats.tiles += w.total_tiles;
        c->stats.last_kernel_grid = (uint64_t)grid;
        c->work_in_flight = true;
    }
    return HPL_OK;
}

int launch_reduce_tasks(hpl_ctx* c, ReduceOp& op, std::vector<PlannedReduceTask>& tasks) {
    if (tasks.empty()) return HPL_OK;
    int max_level = 0;
    for (auto& t : tasks) max_level = std::max(max_level, t.level);
    for (int level = 1; level <= max_level; ++level) {
        std::vector<std::pair<ReduceOp*, PlannedReduceTask*>> lv;
        for (auto& t : tasks)
            if (t.level == level) lv.push_back({&op, &t});
        int rc = launch_reduce_group(c, lv, op.in_dtype == HPL_BF16);
        if (rc != HPL_OK) return rc;
    }
    return HPL_OK;
}

// A position's own object changed, or the position disappeared: its buffer is void, and so is, in every
// ancestor, whatever was merged from the child on that path onwards.  What an ancestor had merged BEFORE that
// child (its earlier operands) is untouched and kept -- healthy chunks are not redone.
void apply_invalidation(hpl_ctx* c, ReduceOp& op, const ReduceInvalidation& inv) {
    const int k = op.sched->k();
    ReduceTreeSchedule& s = *op.sched;
    if (inv.shrank) {
        // the positions that disappeared give their buffers back (once nothing enqueued can still read them)
        bool waited = false;
        for (int q = k; q < (int)op.partial_key.size(); ++q) {
            if (op.partial_key[q] == 0) continue;
            Object* po = find(c, op.partial_key[q]);
            if (!po) continue;
            if (!waited && c->device && (c->work_in_flight || c->copy_pending)) {
                cudaStreamSynchronize(c->copy_stream);
                cudaStreamSynchronize(c->stream);
                waited = true;
            }
            release_object_memory(c, *po);
            c->objects.erase(op.partial_key[q]);
        }
        op.merged.resize(k);
        op.partial_key.resize(k, 0);
    }
    for (int x : inv.touched) {
        if (x < 0) continue;
        if (x < k) op.merged[x].clear();
        for (int child = x, u = s.parent(x); u >= 0; child = u, u = s.parent(u))
            if (u < k) op.merged[u].truncate_above(operand_index_of_child(s, u, child));
    }
}

}  // namespace hpl
