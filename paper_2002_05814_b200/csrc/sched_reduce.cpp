#include "sched_reduce.h"

#include <algorithm>
#include <cmath>

namespace hpl {

// In-order of the complete d-ary tree, written as a rank computation instead of a walk: the
// traversal of a node is [subtree(child 0)] node [subtree(child 1)] ... [subtree(child d-1)].
static void inorder_rec(int p, int k, int d, std::vector<int>& out) {
    const int64_t c0 = (int64_t)d * p + 1;
    if (c0 < k) inorder_rec((int)c0, k, d, out);
    out.push_back(p);
    for (int j = 1; j < d; ++j) {
        const int64_t c = c0 + j;
        if (c >= k) break;
        inorder_rec((int)c, k, d, out);
    }
}

std::vector<int> generalised_inorder(int k, int d) {
    std::vector<int> out;
    out.reserve(k > 0 ? k : 0);
    if (k <= 0) return out;
    if (d == 1) {  // a chain: deepest node first (avoids deep recursion)
        for (int p = k - 1; p >= 0; --p) out.push_back(p);
        return out;
    }
    inorder_rec(0, k, d, out);
    return out;
}

int choose_reduce_degree(int n, double size_bytes, double latency_s, double bandwidth_bytes_per_s) {
    if (n <= 1) return 1;
    const double chain = n * latency_s + size_bytes / bandwidth_bytes_per_s;
    const double binary = latency_s * std::log2((double)n) + 2.0 * size_bytes / bandwidth_bytes_per_s;
    const double star = latency_s + n * size_bytes / bandwidth_bytes_per_s;   // log_n n = 1
    double best = chain;
    int d = 1;
    if (binary < best) {
        best = binary;
        d = 2;
    }
    if (star < best) d = n;
    return d;
}

ReduceTreeSchedule::ReduceTreeSchedule(const std::vector<int64_t>& srcs, int k, int d)
    : srcs_(srcs), k0_(k), k_(k), d_(d), at_(k, -1) {
    const int n = (int)srcs_.size();
    sorted_.reserve(n);
    for (int i = 0; i < n; ++i) sorted_.emplace_back(srcs_[i], i);
    std::sort(sorted_.begin(), sorted_.end());
    alive_.assign(n, 1);
    arrived_.assign(n, 0);
    pos_.assign(n, -1);
}

int ReduceTreeSchedule::index_of(int64_t obj) const {
    auto it = std::lower_bound(sorted_.begin(), sorted_.end(), std::make_pair(obj, -1));
    return (it != sorted_.end() && it->first == obj) ? it->second : -1;
}

int ReduceTreeSchedule::position_of(int64_t obj) const {
    const int i = index_of(obj);
    return i < 0 ? -1 : pos_[i];
}

bool ReduceTreeSchedule::full() const {
    if (k_ <= 0) return false;
    for (int64_t o : at_)
        if (o < 0) return false;
    return true;
}

int ReduceTreeSchedule::live() const {
    int n = 0;
    for (uint8_t a : alive_) n += a;
    return n;
}

int ReduceTreeSchedule::n_children(int p) const {
    const int64_t c0 = (int64_t)d_ * p + 1;
    if (c0 >= k_) return 0;
    return (int)std::min<int64_t>(d_, k_ - c0);
}

std::vector<int> ReduceTreeSchedule::strict_ancestors(int p) const {
    std::vector<int> a;
    while (p > 0) {
        p = (p - 1) / d_;
        a.push_back(p);
    }
    return a;
}

int ReduceTreeSchedule::first_open() const {
    if (order_k_ != k_) {
        order_ = generalised_inorder(k_, d_);
        order_k_ = k_;
        filled_prefix_ = 0;
    }
    for (; filled_prefix_ < order_.size(); ++filled_prefix_)
        if (at_[order_[filled_prefix_]] < 0) return order_[filled_prefix_];
    return -1;
}

void ReduceTreeSchedule::assign(int64_t obj, int pos) {
    at_[pos] = obj;
    pos_[index_of(obj)] = pos;
    placements_.emplace_back(obj, pos);
}

void ReduceTreeSchedule::arrive(int64_t obj) {
    const int i = index_of(obj);
    if (i < 0 || !alive_[i] || arrived_[i]) return;
    arrived_[i] = 1;
    const int p = first_open();
    if (p < 0)
        spares_.push_back(obj);
    else
        assign(obj, p);
}

void ReduceTreeSchedule::rejoin(int64_t obj) {
    const int i = index_of(obj);
    if (i < 0 || alive_[i]) return;
    alive_[i] = 1;
    arrived_[i] = 0;
}

ReduceInvalidation ReduceTreeSchedule::fail(int64_t obj, int64_t delivered,
                                            const std::function<int64_t(int64_t)>& delivered_of) {
    ReduceInvalidation inv;
    filled_prefix_ = 0;   // a position may open anywhere
    const int i = index_of(obj);
    if (i < 0 || !alive_[i]) return inv;
    alive_[i] = 0;
    auto sp = std::find(spares_.begin(), spares_.end(), obj);
    if (sp != spares_.end()) spares_.erase(sp);
    if (pos_[i] >= 0) {
        const int p = pos_[i];
        pos_[i] = -1;
        at_[p] = -1;
        ++epoch_;
        inv.positions.push_back(p);
        inv.touched.push_back(p);
        if (!spares_.empty()) {
            const int64_t s = spares_.front();
            spares_.erase(spares_.begin());
            assign(s, p);
            ReduceEdit e{epoch_, RED_EDIT_REPLACE, p, obj, s, -1, delivered, 0, strict_ancestors(p)};
            for (int a : e.cleared) inv.positions.push_back(a);
            edits_.push_back(std::move(e));
        } else if (live() >= k_) {
            ReduceEdit e{epoch_, RED_EDIT_HOLE, p, obj, -1, -1, delivered, 0, strict_ancestors(p)};
            for (int a : e.cleared) inv.positions.push_back(a);
            edits_.push_back(std::move(e));
        } else {
            shrink(p, obj, delivered, delivered_of, inv);
        }
    } else if (live() < k_) {
        ++epoch_;
        shrink(-1, -1, 0, delivered_of, inv);
    }
    return inv;
}

void ReduceTreeSchedule::shrink(int p, int64_t old_obj, int64_t hi_failed,
                                const std::function<int64_t(int64_t)>& delivered_of, ReduceInvalidation& inv) {
    const int q = k_ - 1;
    const int64_t moved = at_[q];
    std::vector<int> cleared = p >= 0 ? strict_ancestors(p) : std::vector<int>();
    const std::vector<int> q_anc = strict_ancestors(q);  // in the tree before it shrinks
    --k_;
    at_.pop_back();
    inv.shrank = true;
    inv.touched.push_back(q);
    int64_t dest = -1, hi_moved = 0, moved_from = -1, new_obj = -1;
    if (q != p && moved >= 0) {
        pos_[index_of(moved)] = -1;
        dest = p >= 0 ? p : first_open();
        hi_moved = delivered_of ? delivered_of(moved) : 0;
        moved_from = q;
        for (int a : q_anc)
            if (std::find(cleared.begin(), cleared.end(), a) == cleared.end()) cleared.push_back(a);
        assign(moved, (int)dest);
        new_obj = moved;
        inv.touched.push_back((int)dest);
        if (std::find(inv.positions.begin(), inv.positions.end(), (int)dest) == inv.positions.end())
            inv.positions.push_back((int)dest);
    } else {
        dest = (p >= 0 && p != q) ? p : -1;
    }
    for (int a : cleared)
        if (std::find(inv.positions.begin(), inv.positions.end(), a) == inv.positions.end()) inv.positions.push_back(a);
    // the parent of the removed position lost a child even if nothing moved
    for (int a : q_anc)
        if (std::find(inv.positions.begin(), inv.positions.end(), a) == inv.positions.end()) inv.positions.push_back(a);
    edits_.push_back(ReduceEdit{epoch_, RED_EDIT_SHRINK, dest, old_obj, new_obj, moved_from, hi_failed, hi_moved,
                                std::move(cleared)});
}

void ReduceTreeSchedule::dump(int64_t target, std::vector<int64_t>& w) const {
    w.clear();
    w.insert(w.end(), {0x48504C52, target, (int64_t)srcs_.size(), k0_, k_, d_, (int64_t)placements_.size()});
    for (auto& pl : placements_) {
        w.push_back(pl.first);
        w.push_back(pl.second);
    }
    for (int64_t o : at_) w.push_back(o);
    for (int p = 0; p < k_; ++p) w.push_back(parent(p));
    w.push_back((int64_t)spares_.size());
    for (int64_t s : spares_) w.push_back(s);
    w.push_back((int64_t)edits_.size());
    for (auto& e : edits_) {
        w.insert(w.end(), {e.epoch, e.kind, e.pos, e.old_obj, e.new_obj, e.moved_from, e.hi_failed, e.hi_moved,
                           (int64_t)e.cleared.size()});
        for (int c : e.cleared) w.push_back(c);
    }
}

}  // namespace hpl
