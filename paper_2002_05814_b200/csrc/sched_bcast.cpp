#include "sched_bcast.h"

#include <algorithm>

namespace hpl {

BroadcastTreeSchedule::BroadcastTreeSchedule(int64_t src_obj, int64_t n_chunks, int d, int64_t tau)
    : src_(src_obj), C_(n_chunks), tau_(tau), d_(d) {
    BcastLocation s;
    s.obj = src_obj;
    s.slots = d;
    s.t_join = 0;
    locs_.push_back(s);
    index_[src_obj] = 0;
}

int BroadcastTreeSchedule::index_of(int64_t obj) const {
    auto it = index_.find(obj);
    return it == index_.end() ? -1 : it->second;
}

bool BroadcastTreeSchedule::is_waiting(int idx) const {
    return std::find(waiting_.begin(), waiting_.end(), idx) != waiting_.end();
}

void BroadcastTreeSchedule::release(std::vector<int>& v, int x) {
    auto it = std::find(v.begin(), v.end(), x);
    if (it != v.end()) v.erase(it);
}

void BroadcastTreeSchedule::source_progress(int64_t t, int64_t have) {
    advance(t);
    BcastLocation& s = locs_[0];
    s.have = std::max(s.have, have);
    if (s.have >= C_ && !s.complete) {
        s.complete = true;
        s.t_complete = t;
    }
    for (size_t i = 0; i < locs_[0].receivers.size(); ++i) try_start(locs_[0].receivers[i], t);
}

void BroadcastTreeSchedule::advance(int64_t t) {
    while (!heap_.empty() && heap_.top().t <= t) {
        const Landing l = heap_.top();
        heap_.pop();
        BcastLocation& r = locs_[l.order];
        if (r.landing < 0 || r.token != l.token) continue;  // that transfer was cancelled
        land(l.order, l.t);
    }
    now_ = std::max(now_, t);
}

void BroadcastTreeSchedule::try_start(int ri, int64_t t) {
    BcastLocation& r = locs_[ri];
    if (!r.alive || r.complete || r.landing >= 0 || r.sender < 0) return;
    if (locs_[r.sender].have > r.have) {
        r.landing = t + tau_;
        r.token = ++next_token_;
        heap_.push(Landing{r.landing, ri, r.token});
    }
}

void BroadcastTreeSchedule::land(int ri, int64_t t) {
    locs_[ri].landing = -1;
    locs_[ri].have += 1;
    if (locs_[ri].have >= C_) {
        locs_[ri].complete = true;
        locs_[ri].t_complete = t;
        const int s = locs_[ri].sender;
        if (s >= 0) {
            release(locs_[s].receivers, ri);
            if (locs_[s].alive) locs_[s].slots += 1;
        }
        locs_[ri].sender = -1;
        serve_waiting(t);
    } else {
        try_start(ri, t);
    }
    // (try_start never changes a receiver list, so no copy is needed)
    for (size_t i = 0; i < locs_[ri].receivers.size(); ++i) try_start(locs_[ri].receivers[i], t);
}

bool BroadcastTreeSchedule::depends_on(int cand, int root) const {
    for (int x = cand; x >= 0; x = locs_[x].sender)
        if (x == root) return true;
    return false;
}

int BroadcastTreeSchedule::choose(int r) const {
    int best = -1;
    for (int i = 0; i < (int)locs_.size(); ++i) {
        const BcastLocation& l = locs_[i];
        if (!l.alive || i == r || l.slots <= 0) continue;
        if (depends_on(i, r)) continue;
        if (l.complete) return i;
        if (best < 0) best = i;
    }
    return best;
}

void BroadcastTreeSchedule::attach(int r, int s, int64_t t) {
    locs_[s].slots -= 1;
    locs_[s].receivers.push_back(r);
    locs_[r].sender = s;
    locs_[r].last_sender = s;
    locs_[r].start_chunk = locs_[r].have;
    try_start(r, t);
}

void BroadcastTreeSchedule::serve_waiting(int64_t t) {
    bool progressed = true;
    while (progressed) {
        progressed = false;
        for (size_t i = 0; i < waiting_.size(); ++i) {
            const int r = waiting_[i];
            const int s = choose(r);
            if (s >= 0) {
                waiting_.erase(waiting_.begin() + i);
                attach(r, s, t);
                edits_.push_back({++epoch_, BC_EDIT_REPARENT, locs_[r].obj, -1, locs_[s].obj, locs_[r].have, t});
                progressed = true;
                break;
            }
        }
    }
}

void BroadcastTreeSchedule::join(int64_t t, int64_t dst_obj) {
    advance(t);
    {
        auto it = index_.find(dst_obj);
        if (it != index_.end() && locs_[it->second].alive) return;  // a request for this copy is already in flight
        // (a receiver whose worker failed and was rebuilt asks again: a new location)
    }
    BcastLocation r;
    r.obj = dst_obj;
    r.slots = d_;
    r.t_join = t;
    const int ri = (int)locs_.size();
    locs_.push_back(r);
    index_[dst_obj] = ri;
    const int s = choose(ri);
    if (s < 0) {
        waiting_.push_back(ri);
    } else {
        locs_[ri].first_sender_obj = locs_[s].obj;
        attach(ri, s, t);
    }
    serve_waiting(t);
}

void BroadcastTreeSchedule::fail(int64_t t, const std::vector<int64_t>& objs) {
    advance(t);
    std::vector<int> gone;
    for (int64_t o : objs) {
        const int i = index_of(o);
        if (i >= 0 && locs_[i].alive) gone.push_back(i);
    }
    std::sort(gone.begin(), gone.end());
    std::vector<int> orphans;
    for (int g : gone) {
        BcastLocation& L = locs_[g];
        L.alive = false;
        L.landing = -1;
        release(waiting_, g);
        const int s = L.sender;
        if (s >= 0) {
            release(locs_[s].receivers, g);
            if (locs_[s].alive) locs_[s].slots += 1;
            L.sender = -1;
        }
        edits_.push_back({++epoch_, BC_EDIT_LEFT, L.obj, s >= 0 ? locs_[s].obj : -1, -1, L.have, t});
        for (int c : L.receivers) orphans.push_back(c);
        L.receivers.clear();
    }
    std::vector<int> live;
    for (int o : orphans)
        if (locs_[o].alive) live.push_back(o);
    std::sort(live.begin(), live.end());
    std::vector<int> olds;
    for (int o : live) {  // every orphan first loses its sender and its chunk in flight ...
        locs_[o].landing = -1;
        olds.push_back(locs_[o].sender);
        locs_[o].sender = -1;
    }
    for (size_t i = 0; i < live.size(); ++i) {  // ... then each, oldest first, asks the directory again
        const int o = live[i];
        const int s = choose(o);
        ++epoch_;
        const int64_t old_obj = olds[i] >= 0 ? locs_[olds[i]].obj : -1;
        if (s < 0) {
            waiting_.push_back(o);
            edits_.push_back({epoch_, BC_EDIT_WAIT, locs_[o].obj, old_obj, -1, locs_[o].have, t});
        } else {
            attach(o, s, t);
            edits_.push_back({epoch_, BC_EDIT_REPARENT, locs_[o].obj, old_obj, locs_[s].obj, locs_[o].have, t});
        }
    }
    serve_waiting(t);
}

bool BroadcastTreeSchedule::run_until_complete(int64_t obj) {
    const int i = index_of(obj);
    if (i < 0) return false;
    while (!locs_[i].complete && !heap_.empty()) advance(heap_.top().t);
    return locs_[i].complete;
}

void BroadcastTreeSchedule::dump(std::vector<int64_t>& w) const {
    w.clear();
    w.insert(w.end(), {0x48504C42, src_, d_, C_, tau_, now_, (int64_t)locs_.size() - 1});
    for (size_t i = 1; i < locs_.size(); ++i) {
        const BcastLocation& r = locs_[i];
        w.insert(w.end(), {r.obj, r.first_sender_obj, r.sender >= 0 ? locs_[r.sender].obj : -1, r.start_chunk, r.t_join,
                           r.have, r.alive ? 1 : 0, r.t_complete});
    }
    w.push_back((int64_t)edits_.size());
    for (auto& e : edits_) w.insert(w.end(), e.begin(), e.end());
}

}  // namespace hpl
