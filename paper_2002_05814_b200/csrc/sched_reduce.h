// Reduce schedule builder (host side, no CUDA): tree shape, arrival-order placement, k-of-m
// selection and failure edits of Hoplite's Reduce (arXiv 2002.05814, Sections 3.4.2 and 3.5.2).
//
// The tree over k objects is the complete d-ary tree on positions 0..k-1 in level order.  An
// arriving object takes the first open position of the generalised in-order traversal (first
// child's subtree, the node, then the other children's subtrees).  Arrivals beyond k wait as
// spares.  A failed member leaves at once: the oldest spare replaces it, else the position stays
// open for the next arrival while enough live sources remain, else the tree shrinks by its last
// position and the object there (if any) moves into the opening.  Ancestors of every touched
// position lose their partial results.
#pragma once
#include <cstdint>
#include <functional>
#include <vector>

namespace hpl {

enum { RED_EDIT_REPLACE = 1, RED_EDIT_HOLE = 2, RED_EDIT_SHRINK = 3 };

struct ReduceEdit {
    int64_t epoch, kind, pos, old_obj, new_obj, moved_from, hi_failed, hi_moved;
    std::vector<int> cleared;
};

// What an edit means for materialised results: positions whose own partial must be recomputed.
struct ReduceInvalidation {
    std::vector<int> positions;   // includes the vacated position itself and all cleared ancestors
    std::vector<int> touched;     // positions whose own object changed or that disappeared (old numbering)
    bool shrank = false;          // the last position disappeared
};

class ReduceTreeSchedule {
public:
    ReduceTreeSchedule(const std::vector<int64_t>& srcs, int k, int d);

    int k() const { return k_; }
    int k_requested() const { return k0_; }
    int d() const { return d_; }
    int64_t object_at(int pos) const { return at_[pos]; }
    int position_of(int64_t obj) const;
    bool has_source(int64_t obj) const { return index_of(obj) >= 0; }
    bool full() const;
    int live() const;
    const std::vector<int64_t>& sources() const { return srcs_; }

    int parent(int p) const { return p == 0 ? -1 : (p - 1) / d_; }
    int first_child(int p) const { return d_ * p + 1; }
    int n_children(int p) const;
    bool is_leaf(int p) const { return (int64_t)d_ * p + 1 >= k_; }

    // events; each returns the positions whose materialised results are no longer valid
    void arrive(int64_t obj);
    void rejoin(int64_t obj);   // a failed source was reconstructed: a future again, a new arrival when put again
    ReduceInvalidation fail(int64_t obj, int64_t delivered_chunks, const std::function<int64_t(int64_t)>& delivered_of);

    void dump(int64_t target, std::vector<int64_t>& w) const;

private:
    int first_open() const;
    void assign(int64_t obj, int pos);
    void shrink(int p, int64_t old_obj, int64_t hi_failed, const std::function<int64_t(int64_t)>& delivered_of,
                ReduceInvalidation& inv);
    std::vector<int> strict_ancestors(int p) const;

    std::vector<int64_t> srcs_;
    int k0_, k_, d_;
    int64_t epoch_ = 0;
    // per source, by its index in srcs_ (found through the sorted list: no allocation per source, per event)
    int index_of(int64_t obj) const;
    std::vector<std::pair<int64_t, int>> sorted_;   // (object id, index in srcs_)
    std::vector<uint8_t> alive_, arrived_;
    std::vector<int> pos_;                          // position in the tree, -1 = none
    std::vector<int64_t> at_;
    std::vector<int64_t> spares_;
    std::vector<std::pair<int64_t, int>> placements_;
    std::vector<ReduceEdit> edits_;
    // the in-order of the current tree, kept between arrivals, and how far it is known to be filled (reset by every
    // event that can open a position)
    mutable std::vector<int> order_;
    mutable int order_k_ = -1;
    mutable size_t filled_prefix_ = 0;
};

// Eq. 1 / Section 4: the degree among 1, 2 and n with the smallest estimated reduce time (ties: the smaller).
int choose_reduce_degree(int n, double size_bytes, double latency_s, double bandwidth_bytes_per_s);

// Positions of the complete d-ary tree on k nodes in generalised in-order.
std::vector<int> generalised_inorder(int k, int d);

}  // namespace hpl
