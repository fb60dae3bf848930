// Broadcast planner: which receivers can be served now, from which copy, as fan-out tasks.
#include "context.h"

namespace hpl {

int plan_bcast(hpl_ctx* c, BcastOp& op, std::vector<PlannedFanout>& tasks) {
    BroadcastTreeSchedule& s = *op.sched;
    const auto& locs = s.locations();
    op.phys_have.resize(locs.size(), 0);
    Object* src = find(c, op.src);
    if (!src) return HPL_OK;
    const uint32_t C = src->C;
    uint32_t src_landed = 0, src_avail = 0;
    if (src->alive && src->ptr && src->row >= 0) {
        if (src->kind == OBJ_TARGET) {   // reduce followed by broadcast: the source is a Reduce output
            const uint64_t n = produced_elems(c, *src);   // fp32 elements -> chunks of the broadcast (bytes of the object)
            src_landed = src_avail = n * 4 >= src->bytes ? C : (uint32_t)(n * 4 / c->cfg.chunk_bytes);
        } else {
            src_landed = std::min(published_chunks(c, *src), src->landed);
            src_avail = c->cfg.plan_ahead ? C : src_landed;
        }
    }
    std::vector<int64_t> pre(op.phys_have);  // what every copy holds before this pass
    pre[0] = src_avail;
    std::vector<char> usable_v(locs.size(), 0);   // copies whose buffer may be read or written now
    usable_v[0] = src->alive && src->ptr != nullptr;
    bool any_pending = false;
    for (size_t x = 1; x < locs.size(); ++x) {
        if (!locs[x].alive) continue;
        Object* o = find(c, locs[x].obj);
        usable_v[x] = o && o->alive && o->ptr && o->row >= 0;
        if (usable_v[x] && op.phys_have[x] < (int64_t)C) any_pending = true;
    }
    if (!any_pending) return HPL_OK;
    auto usable = [&](int x) { return usable_v[x] != 0; };
    std::vector<uint32_t> bp = {0u, src_avail};
    for (size_t i = 1; i < locs.size(); ++i) bp.push_back((uint32_t)pre[i]);
    std::sort(bp.begin(), bp.end());
    bp.erase(std::unique(bp.begin(), bp.end()), bp.end());

    std::vector<char> stuck(locs.size(), 0);
    for (size_t bi = 0; bi + 1 < bp.size(); ++bi) {
        const uint32_t a = bp[bi], b = bp[bi + 1];
        std::map<int, std::vector<int>> groups;  // read location (and, in worker-per-GPU mode, hop depth) -> receivers
        if (c->world > 1) {
            // worker-per-GPU mode: bytes cross the interconnect along the tree's edges only -- a receiver is served by
            // its own sender (whose rank pushes), from a copy that holds the interval already or that is itself
            // served in this plan, one hop (level) earlier
            std::vector<int> depth(locs.size(), -1);   // hops of this plan after which the location holds [a, b)
            for (size_t x = 0; x < locs.size(); ++x)
                if (usable((int)x) && pre[x] >= (int64_t)b) depth[x] = 0;
            bool progressed = true;
            while (progressed) {
                progressed = false;
                for (int r = 1; r < (int)locs.size(); ++r) {
                    if (stuck[r] || !usable(r) || locs[r].last_sender < 0 || depth[r] >= 0) continue;
                    if (op.phys_have[r] != (int64_t)a) continue;
                    const int x = locs[r].last_sender;
                    if (!usable(x) || depth[x] < 0) continue;
                    depth[r] = depth[x] + 1;
                    groups[x * 4096 + depth[r]].push_back(r);
                    c->journal.b.push_back({op.src, r, op.phys_have[r], c->batch_tag});
                    op.phys_have[r] = b;
                    progressed = true;
                }
            }
            for (int r = 1; r < (int)locs.size(); ++r)
                if (usable(r) && op.phys_have[r] == (int64_t)a && depth[r] < 0) stuck[r] = 1;
        }
        for (int r = 1; r < (int)locs.size() && c->world <= 1; ++r) {
            if (stuck[r] || !usable(r) || locs[r].last_sender < 0) continue;
            if (op.phys_have[r] != (int64_t)a) continue;  // needs this interval next
            int loc = -1;
            for (int x = locs[r].last_sender, hops = 0; x >= 0 && hops <= (int)locs.size(); x = locs[x].last_sender, ++hops) {
                if (usable(x) && pre[x] >= (int64_t)b) {
                    loc = x;
                    break;
                }
                if (x == 0) break;
            }
            if (loc < 0) {
                for (int x = 0; x < (int)locs.size(); ++x)
                    if (x != r && usable(x) && pre[x] >= (int64_t)b) {
                        loc = x;
                        break;
                    }
            }
            if (loc < 0) {
                stuck[r] = 1;
                continue;
            }
            groups[loc].push_back(r);
            c->journal.b.push_back({op.src, r, op.phys_have[r], c->batch_tag});
            op.phys_have[r] = b;
        }
        for (auto& g : groups) {
            const int loc = c->world > 1 ? g.first / 4096 : g.first;
            const int level = c->world > 1 ? g.first % 4096 : 1;
            const bool poll = (loc == 0) && (src_landed < b);
            bool merged = false;
            for (auto& prev : tasks) {
                if (prev.loc == loc && prev.level == level && prev.b == a && prev.poll == poll && prev.dst == g.second) {
                    prev.b = b;
                    merged = true;
                    break;
                }
            }
            if (!merged) {
                PlannedFanout t{loc, a, b, poll, level, g.second};
                tasks.push_back(std::move(t));
            }
        }
    }
    return HPL_OK;
}

// Packs fan-out tasks (of one broadcast, or of several small ones) into waves and launches them.
int launch_fanout_group(hpl_ctx* c, std::vector<std::pair<BcastOp*, PlannedFanout>>& tasks) {
    if (tasks.empty()) return HPL_OK;
    const uint64_t chunk_bytes = c->cfg.chunk_bytes;
    size_t i = 0;
    while (i < tasks.size()) {
        static thread_local FanoutWave w;
        w.dir = c->d_dir;
        w.status = nullptr;
        w.budget_ns = c->cfg.poll_budget_ns;
        w.n_tasks = 0;
        w.total_tiles = 0;
        uint32_t n_dst = 0;
        while (i < tasks.size() && w.n_tasks < (uint32_t)kMaxFanoutTasks) {
            if (tasks[i].second.dst.size() > (size_t)kMaxFanoutDst) {
                // more receivers than one task holds: split the receiver list
                std::pair<BcastOp*, PlannedFanout> rest = tasks[i];
                rest.second.dst.assign(tasks[i].second.dst.begin() + kMaxFanoutDst, tasks[i].second.dst.end());
                tasks[i].second.dst.resize(kMaxFanoutDst);
                tasks.insert(tasks.begin() + i + 1, rest);
                continue;
            }
            if (n_dst + tasks[i].second.dst.size() > (size_t)kMaxFanoutDst) break;
            BcastOp& op = *tasks[i].first;
            PlannedFanout& tt = tasks[i].second;
            Object* src = find(c, op.src);
            const auto& locs = op.sched->locations();
            const uint32_t tpc = (uint32_t)((std::min<uint64_t>(chunk_bytes, src->bytes) + kFanoutTileBytes - 1) / kFanoutTileBytes);
            FanoutTask& d = w.tasks[w.n_tasks++];
            Object* lo = tt.loc == 0 ? src : find(c, locs[tt.loc].obj);
            d.src_row = (uint32_t)lo->row;
            d.src_ptr = (unsigned long long)(uintptr_t)lo->ptr;
            d.c_begin = tt.a;
            d.c_end = tt.b;
            d.tiles_per_chunk = tpc;
            d.tile_bytes = kFanoutTileBytes;
            d.tile_begin = w.total_tiles;
            d.dst_begin = n_dst;
            d.n_dst = (uint32_t)tt.dst.size();
            d.poll = tt.poll ? 1u : 0u;
            if (tt.poll) c->polling_in_flight = true;
            d.bytes = src->bytes;
            d.chunk_bytes = chunk_bytes;
            for (int r : tt.dst) {
                const Object* ro = find(c, locs[r].obj);
                w.dst_rows[n_dst] = (uint32_t)ro->row;
                w.dst_ptrs[n_dst++] = (unsigned long long)(uintptr_t)ro->ptr;
            }
            w.total_tiles += (tt.b - tt.a) * tpc;
            const uint64_t b_lo = (uint64_t)tt.a * chunk_bytes, b_hi = std::min<uint64_t>((uint64_t)tt.b * chunk_bytes, src->bytes);
            c->stats.bytes_read_planned += b_hi - b_lo;
            c->stats.bytes_written_planned += (b_hi - b_lo) * tt.dst.size();
            c->stats.fanout_tasks++;
            ++i;
        }
        if (w.n_tasks == 0) return HPL_ERR_INVALID;
        if (!c->device) {   // schedule-only context: planned and counted, not run
            c->stats.kernel_launches++;
            c->stats.fanout_launches++;
            c->stats.tiles += w.total_tiles;
            continue;
        }
        if (c->occ_fanout == 0) c->occ_fanout = fanout_ctas_per_sm();
        const uint32_t tb = spread_tile_bytes(w.total_tiles, (uint64_t)c->n_sm * c->occ_fanout, kFanoutTileBytes, 512, 4096);
        if (tb != (uint32_t)kFanoutTileBytes) {
            w.total_tiles = 0;
            for (uint32_t q = 0; q < w.n_tasks; ++q) {
                FanoutTask& d = w.tasks[q];
                d.tile_bytes = tb;
                d.tiles_per_chunk = (uint32_t)((std::min<uint64_t>(d.chunk_bytes, d.bytes) + tb - 1) / tb);
                d.tile_begin = w.total_tiles;
                w.total_tiles += (d.c_end - d.c_begin) * d.tiles_per_chunk;
            }
        }
        int grid = (int)std::min<uint64_t>(w.total_tiles, (uint64_t)c->n_sm * c->occ_fanout);
        if (grid < 1) grid = 1;
        if (flush_directory(c) != HPL_OK) return HPL_ERR_CUDA;
        bool polls = kDebugBounds;   // (the bounds-checking build reads the directory in every wave, and may record an error)
        for (uint32_t q = 0; q < w.n_tasks; ++q) polls = polls || w.tasks[q].poll;
        if (polls && order_main_after_control(c) != HPL_OK) return HPL_ERR_CUDA;   // the counter it waits on is a row of the directory
        if (kDebugBounds) c->polling_in_flight = true;
        w.status = next_wave_status(c);
        {
            LaunchTimer timer(c, 1);
            if (launch_fanout_wave(w, grid, c->stream) != 0) return HPL_ERR_CUDA;
        }
        c->stats.kernel_launches++;
        c->stats.fanout_launches++;
        c->stats.tiles += w.total_tiles;
        c->stats.last_kernel_grid = (uint64_t)grid;
        c->work_in_flight = true;
    }
    return HPL_OK;
}

int launch_fanout_tasks(hpl_ctx* c, BcastOp& op, std::vector<PlannedFanout>& tasks) {
    std::vector<std::pair<BcastOp*, PlannedFanout>> g;
    for (auto& t : tasks) g.push_back({&op, std::move(t)});
    return launch_fanout_group(c, g);
}

}  // namespace hpl
