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

// Chunks a receiver holds at time t in the closed form: those with b + (c + 1) tau <= t.
int64_t BroadcastTreeSchedule::held_at(const BcastLocation& l, int64_t t) const {
    if (l.complete) return C_;
    if (t <= l.b) return 0;
    return std::min<int64_t>(C_, (t - l.b) / tau_);
}

// Leaves the closed form: writes down, for the current time, what every receiver holds and which chunk is on
// its way, exactly as the event simulation would have it, and goes on chunk by chunk.
void BroadcastTreeSchedule::to_events() {
    if (!closed_form_) return;
    closed_form_ = false;
    for (size_t i = 1; i < locs_.size(); ++i)
        if (locs_[i].alive && !locs_[i].complete) locs_[i].have = held_at(locs_[i], now_);
    for (size_t i = 1; i < locs_.size(); ++i) {
        BcastLocation& r = locs_[i];
        if (!r.alive || r.complete || r.sender < 0) continue;
        if (locs_[r.sender].have > r.have) {   // its next chunk is on its way
            r.landing = r.b + (r.have + 1) * tau_;
            r.token = ++next_token_;
            heap_.push(Landing{r.landing, (int)i, r.token});
        }
    }
    while (!completions_.empty()) completions_.pop();
}

void BroadcastTreeSchedule::complete_location(int ri, int64_t t) {
    locs_[ri].have = C_;
    locs_[ri].complete = true;
    locs_[ri].t_complete = t;
    const int s = locs_[ri].sender;
    if (s >= 0) {
        release(locs_[s].receivers, ri);
        if (locs_[s].alive) locs_[s].slots += 1;
    }
    locs_[ri].sender = -1;
}

void BroadcastTreeSchedule::source_progress(int64_t t, int64_t have) {
    if (closed_form_ && locs_.size() > 1 && have < C_) to_events();   // (cannot happen: receivers only join a complete source here)
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
    if (closed_form_) {
        while (!completions_.empty() && completions_.top().first <= t) {
            const Completion cmp = completions_.top();
            completions_.pop();
            complete_location(cmp.second, cmp.first);   // nobody waits in the closed form: a freed slot is just a count
        }
        now_ = std::max(now_, t);
        return;
    }
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
        complete_location(ri, t);
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
    if (closed_form_ && !locs_[0].complete) to_events();   // a source that is still being put: chunk by chunk
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
    if (closed_form_ && s >= 0) {
        // evenly spaced landings: chunk c at b + (c + 1) tau, complete at b + C tau
        BcastLocation& r = locs_[ri];
        r.first_sender_obj = locs_[s].obj;
        locs_[s].slots -= 1;
        locs_[s].receivers.push_back(ri);
        r.sender = r.last_sender = s;
        r.start_chunk = 0;
        r.b = (s == 0 || locs_[s].complete) ? t : std::max(locs_[s].b + tau_, t);
        completions_.push(Completion(r.b + C_ * tau_, ri));
        return;
    }
    to_events();   // a receiver that has to wait: chunk by chunk from here on
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
    to_events();
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
    if (closed_form_) {
        if (!locs_[i].complete && locs_[i].alive) advance(locs_[i].b + C_ * tau_);
        return locs_[i].complete;
    }
    while (!locs_[i].complete && !heap_.empty()) advance(heap_.top().t);
    return locs_[i].complete;
}

void BroadcastTreeSchedule::dump(std::vector<int64_t>& w) const {
    w.clear();
    w.insert(w.end(), {0x48504C42, src_, d_, C_, tau_, now_, (int64_t)locs_.size() - 1});
    for (size_t i = 1; i < locs_.size(); ++i) {
        const BcastLocation& r = locs_[i];
        w.insert(w.end(), {r.obj, r.first_sender_obj, r.sender >= 0 ? locs_[r.sender].obj : -1, r.start_chunk, r.t_join,
                           closed_form_ ? held_at(r, now_) : r.have, r.alive ? 1 : 0, r.t_complete});
    }
    w.push_back((int64_t)edits_.size());
    for (auto& e : edits_) w.insert(w.end(), e.begin(), e.end());
}

}  // namespace hpl
