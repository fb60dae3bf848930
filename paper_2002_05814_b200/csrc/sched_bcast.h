// Broadcast schedule builder (host side, no CUDA): receiver-driven tree formation and failover
// of Hoplite's broadcast (arXiv 2002.05814, Sections 3.4.1 and 3.5.1), in virtual time.
//
// Every copy of the object is a "location": the source first, then the receivers in join
// order.  A joining receiver is given the oldest complete location with a free send slot, else
// the oldest partial one; the slot is held until the receiver has the whole object.  One chunk
// crosses one edge in `tau` ns; a receiver fetches chunks in order, one at a time, each as soon
// as its sender holds it.  When a location fails, the receivers it was sending to ask again
// (candidates that fetch, directly or not, from the asker are not eligible) and resume from
// the chunks they hold.
//
// Two engines compute the same virtual-time model.  While the source was complete before the first
// receiver joined and nothing has failed or had to wait, every receiver's chunks land at evenly spaced
// times, L_r(c) = b_r + (c + 1) tau with b_r = max(b_sender + tau, t_join) (by induction over
// avail_r(c) = max(avail_sender(c), avail_r(c - 1), t_join) + tau): only the completions are events, and
// the chunks held at a time follow from b_r.  Anything else -- a source that is still being put, a
// failure, a receiver without a sender -- first turns that state into the per-chunk event simulation
// (chunks held, transfer in flight) and continues there.
#pragma once
#include <cstdint>
#include <queue>
#include <unordered_map>
#include <vector>

namespace hpl {

enum { BC_EDIT_REPARENT = 1, BC_EDIT_WAIT = 2, BC_EDIT_LEFT = 3 };

struct BcastLocation {
    int64_t obj = -1;
    int64_t have = 0;          // chunks held in virtual time
    bool complete = false;
    bool alive = true;
    int slots = 0;
    int sender = -1;           // index into the location list, -1 none
    int last_sender = -1;      // the most recent sender ever attached (kept after completion)
    int64_t first_sender_obj = -1;
    int64_t start_chunk = 0;
    int64_t t_join = -1, t_complete = -1;
    int64_t landing = -1;      // time the chunk in flight lands, -1 none
    uint64_t token = 0;        // identifies the transfer in flight
    int64_t b = 0;             // closed form: chunk c lands at b + (c + 1) tau
    std::vector<int> receivers;
};

class BroadcastTreeSchedule {
public:
    BroadcastTreeSchedule(int64_t src_obj, int64_t n_chunks, int d, int64_t tau);

    void source_progress(int64_t t, int64_t have);
    void advance(int64_t t);
    void join(int64_t t, int64_t dst_obj);
    void fail(int64_t t, const std::vector<int64_t>& objs);
    // Lets virtual time run until `obj` is complete; false if no pending transfer can complete it.
    bool run_until_complete(int64_t obj);

    int64_t now() const { return now_; }
    int index_of(int64_t obj) const;
    const std::vector<BcastLocation>& locations() const { return locs_; }
    bool is_waiting(int idx) const;
    void dump(std::vector<int64_t>& w) const;

private:
    struct Landing {
        int64_t t;
        int order;
        uint64_t token;
        bool operator>(const Landing& o) const { return t != o.t ? t > o.t : (order != o.order ? order > o.order : token > o.token); }
    };
    void try_start(int r, int64_t t);
    void land(int r, int64_t t);
    int choose(int r) const;
    bool depends_on(int cand, int root) const;
    void attach(int r, int s, int64_t t);
    void serve_waiting(int64_t t);
    void release(std::vector<int>& v, int x);
    void complete_location(int r, int64_t t);
    int64_t held_at(const BcastLocation& l, int64_t t) const;
    void to_events();

    int64_t src_, C_, tau_, now_ = 0, epoch_ = 0;
    int d_;
    uint64_t next_token_ = 0;
    std::vector<BcastLocation> locs_;
    std::unordered_map<int64_t, int> index_;
    std::vector<int> waiting_;
    std::vector<std::vector<int64_t>> edits_;
    std::priority_queue<Landing, std::vector<Landing>, std::greater<Landing>> heap_;
    bool closed_form_ = true;                            // evenly spaced landings: only completions are events
    typedef std::pair<int64_t, int> Completion;          // (time, location)
    std::priority_queue<Completion, std::vector<Completion>, std::greater<Completion>> completions_;
};

}  // namespace hpl
