// Internal declarations shared by the host-side translation units of the library: the context, the
// object table, the per-collective execution state, and the helpers that touch the device directory.
#pragma once
#include <cuda_runtime.h>

#include <algorithm>
#include <cstddef>
#include <cstdlib>
#include <cstring>
#include <map>
#include <memory>
#include <set>
#include <unordered_map>
#include <vector>

#include "../../include/hpl.h"
#include "device_types.h"
#include "sched_bcast.h"
#include "sched_reduce.h"

namespace hpl {

constexpr uint32_t kMaxRows = 4096;
constexpr uint32_t kStatusSlots = 256;   // one error record per wave in flight; beyond that the last one is shared
constexpr uint32_t kMaxChunks = 1u << 20;
constexpr uint64_t kAlign = 256;
constexpr uint32_t kStageRows = 4 * kMaxRows;
constexpr uint64_t kSmallObjectBytes = 64 * 1024;   // Section 3.2's threshold for small objects

// Per tree position: for which chunks how many leading operands of the node (first child, own object, second
// child, ...) have been merged into its result buffer.  All operands merged = the node's result is complete.
struct IntervalMap {  // disjoint, sorted [a, b) -> value > 0
    struct E { uint32_t a, b; int v; };
    std::vector<E> iv;
    void clear() { iv.clear(); }
    int value_at(uint32_t c) const {
        for (auto& x : iv)
            if (x.a <= c && c < x.b) return x.v;
        return 0;
    }
    void set(uint32_t a, uint32_t b, int v) {   // v == 0 erases
        if (a >= b) return;
        std::vector<E> out;
        for (auto& x : iv) {
            if (x.b <= a || b <= x.a) {
                out.push_back(x);
                continue;
            }
            if (x.a < a) out.push_back({x.a, a, x.v});
            if (b < x.b) out.push_back({b, x.b, x.v});
        }
        if (v > 0) out.push_back({a, b, v});
        std::sort(out.begin(), out.end(), [](const E& l, const E& r) { return l.a < r.a; });
        iv.clear();
        for (auto& x : out) {   // join neighbours with the same value
            if (!iv.empty() && iv.back().b == x.a && iv.back().v == x.v)
                iv.back().b = x.b;
            else
                iv.push_back(x);
        }
    }
    void truncate_above(int j) {   // forget everything that has more than j operands merged
        std::vector<E> out;
        for (auto& x : iv)
            if (x.v <= j) out.push_back(x);
        iv.swap(out);
    }
    void breakpoints(std::vector<uint32_t>& bp) const {
        for (auto& x : iv) {
            bp.push_back(x.a);
            bp.push_back(x.b);
        }
    }
    uint32_t full_prefix(int full) const {   // end of the run of complete chunks that starts at chunk 0
        uint32_t end = 0;
        for (auto& x : iv) {
            if (x.a != end || x.v != full) break;
            end = x.b;
        }
        return end;
    }
    bool covers(uint32_t a, uint32_t b, int full) const {
        uint32_t at = a;
        for (auto& x : iv) {
            if (x.b <= at) continue;
            if (x.a > at || x.v != full) return false;
            at = x.b;
            if (at >= b) return true;
        }
        return at >= b;
    }
};

struct Arena {
    uint8_t* base = nullptr;
    uint64_t size = 0, used = 0;
    std::map<uint64_t, uint64_t> free_;  // offset -> length
    void init(void* p, uint64_t n) {
        base = (uint8_t*)p;
        size = n;
        used = 0;
        free_.clear();
        uint64_t off = (kAlign - ((uintptr_t)p % kAlign)) % kAlign;
        if (n > off) free_[off] = n - off;
    }
    void* alloc(uint64_t n) {
        n = (n + kAlign - 1) / kAlign * kAlign;
        for (auto it = free_.begin(); it != free_.end(); ++it) {
            if (it->second >= n) {
                const uint64_t off = it->first, len = it->second;
                free_.erase(it);
                if (len > n) free_[off + n] = len - n;
                used += n;
                sizes_[off] = n;
                return base + off;
            }
        }
        return nullptr;
    }
    void release(void* p) {
        uint64_t off = (uint8_t*)p - base;
        auto s = sizes_.find(off);
        if (s == sizes_.end()) return;
        uint64_t n = s->second;
        sizes_.erase(s);
        used -= n;
        auto next = free_.lower_bound(off);
        if (next != free_.end() && off + n == next->first) {
            n += next->second;
            next = free_.erase(next);
        }
        if (next != free_.begin()) {
            auto prev = std::prev(next);
            if (prev->first + prev->second == off) {
                prev->second += n;
                return;
            }
        }
        free_[off] = n;
    }
    std::map<uint64_t, uint64_t> sizes_;
};

enum ObjKind { OBJ_PLAIN = 0, OBJ_TARGET = 1, OBJ_RECEIVER = 2, OBJ_PARTIAL = 3 };

// The Reduces that name an object as a source (keys of `reduces`), in creation order.  Almost always one: that one
// lives in the object itself, so that a Reduce request allocates nothing per source.
struct ConsumerList {
    uint64_t first = 0;
    bool has_first = false;
    std::vector<uint64_t> rest;
    bool empty() const { return !has_first; }
    void push_back(uint64_t key) {
        if (!has_first) {
            first = key;
            has_first = true;
        } else {
            rest.push_back(key);
        }
    }
    void erase(uint64_t key) {
        if (has_first && first == key) {
            has_first = !rest.empty();
            if (has_first) {
                first = rest.front();
                rest.erase(rest.begin());
            }
        } else {
            rest.erase(std::remove(rest.begin(), rest.end(), key), rest.end());
        }
    }
    template <class F>
    void for_each(F f) const {
        if (!has_first) return;
        f(first);
        for (uint64_t key : rest) f(key);
    }
};

struct Object {
    int64_t id = 0;
    int32_t worker = -1;
    uint64_t bytes = 0;
    int32_t dtype = HPL_F32;
    uint32_t C = 0;
    ObjKind kind = OBJ_PLAIN;
    int64_t op_key = 0;        // receiver: its source id
    void* ptr = nullptr;
    bool lib_owned = false;
    bool from_host = false;
    bool async_counter = false;   // its counter travels on a side stream: kernels poll it until a wait confirms it
    uint64_t ready_bytes = 0;  // published prefix
    uint32_t landed = 0;       // chunks whose counter update is ordered before later launches on the main stream
    bool alive = true;
    bool arrived = false;
    int64_t t_arrival = -1;
    uint64_t seq = 0;          // creation order
    int row = -1;
    int home = 0;              // rank whose GPU holds the bytes (worker-per-GPU mode)
    int pos = -1;              // partial result: its tree position (op_key = the Reduce's target)
    uint64_t last_use = 0;     // partial result: when a planning pass last wrote or read it (eviction order)
    uint64_t last_pass = 0;    //                 and which pass that was
    ConsumerList consumers;    // the Reduces it is a source of
};

struct Journal {  // what was planned since the last successful wait (undone if a device wait expires)
    // tag: the planning pass that made the entry; the waves that pass launches carry the same tag
    struct R { int64_t target; int pos; uint32_t a, b; int old_v; uint64_t tag; };
    struct B { int64_t src; int loc; int64_t old_have; uint64_t tag; };
    std::vector<R> r;
    std::vector<B> b;
    void clear() { r.clear(); b.clear(); }
};

struct PlannedReduceTask {
    int pos;
    int end;      // operands of the position merged once this task has run
    int level;
    uint32_t a, b;
    int n_acc;
    bool poll;
    std::vector<ReduceStep> steps;
    std::vector<unsigned long long> fan;   // buffers of broadcast receivers that take the result from this task (root tasks only)
    std::vector<uint32_t> fan_rows;        // their directory rows
};

struct ReduceOp {
    int64_t target;
    std::unique_ptr<ReduceTreeSchedule> sched;
    int red_op, in_dtype;
    uint64_t elems;
    uint32_t C, chunk_elems;
    uint64_t seq;
    std::vector<IntervalMap> merged;        // per position: chunks -> leading operands merged into its buffer (valid ones only)
    int n_ops(int pos) const { return sched->n_children(pos) + 1; }
    std::vector<int64_t> partial_key;       // per position: internal object id of its partial buffer (0 none)
    bool lost = false;                      // worker-per-GPU mode: the rank that held the output is gone
};

struct BcastOp {
    int64_t src;
    std::unique_ptr<BroadcastTreeSchedule> sched;
    std::vector<int64_t> dsts;
    std::vector<int64_t> phys_have;  // per location index: chunks physically planned (index 0 unused)
    uint64_t seq;
};


struct PlannedFanout {
    int loc;  // location index read from
    uint32_t a, b;
    bool poll;
    int level = 1;  // worker-per-GPU mode: 1 + number of hops of this plan the copy that is read is away from one that holds the interval already
    std::vector<int> dst;  // location indices written
};

}  // namespace hpl

using namespace hpl;   // internal header: the context keeps its C name outside the namespace

struct hpl_ctx {
    hpl_config cfg{};
    cudaStream_t stream = nullptr, copy_stream = nullptr, ctl_stream = nullptr;
    cudaEvent_t copy_ev = nullptr, ctl_ev = nullptr;
    bool device = false;
    bool copy_pending = false;
    bool ctl_pending = false;   // directory updates on the control stream not yet ordered before the main stream
    bool ctl_unconfirmed = false;   // counters of device puts went out on the control stream (plan-ahead) and no wait has confirmed them
    int n_sm = 0;
    uint64_t now = 0, tau = 1, seq = 0;
    int64_t next_internal = -1;  // ids of partial buffers: negative, never visible outside
    hpl::Arena arena;                          // this rank's arena
    int rank = 0, world = 1;
    std::vector<hpl::Arena> peer_arenas;       // worker-per-GPU mode: replicas of the other ranks' allocators (index = rank)
    std::vector<char> rank_alive;
    struct Level {                             // tasks of one dependency level of the current plan, all ranks'
        std::vector<std::pair<ReduceOp*, PlannedReduceTask>> r;
        std::vector<std::pair<BcastOp*, PlannedFanout>> f;
    };
    std::vector<Level> levels;                 // planned, not yet released (worker-per-GPU mode)
    uint64_t use_tick = 0, plan_pass = 0;                      // eviction clock of partial results; planning passes so far
    int64_t planning_target = -1;                              // the Reduce being planned right now (-1 none)
    uint64_t guard_bytes = 0;                                  // testing aid: canary after every arena block
    std::map<void*, std::pair<uint64_t, uint64_t>> guards;     // block -> (offset of its canary, length)
    uint64_t guard_violations = 0;
    DirRow* d_dir = nullptr;
    DirRow* h_dir = nullptr;
    DeviceStatus* d_status = nullptr;
    DeviceStatus* h_status = nullptr;
    uint32_t* h_iota = nullptr;
    DirRow* h_stage = nullptr;           // pinned snapshots of directory rows on their way to the device
    uint32_t stage_cursor = 0;
    std::vector<int> dirty_rows;         // rows changed on the host since the last flush (batched mode)
    std::vector<int> free_rows;
    std::unordered_map<int64_t, Object> objects;
    std::map<uint64_t, ReduceOp> reduces;  // by creation order
    std::map<uint64_t, BcastOp> bcasts;
    std::unordered_map<int64_t, uint64_t> reduce_of_target, bcast_of_src;
    std::set<uint64_t> composed_bcasts;   // keys of the broadcasts whose source is a Reduce output, in creation order
    Journal journal;
    bool work_in_flight = false;
    bool polling_in_flight = false;   // some wave in flight polls progress counters (only those can record an error)
    uint64_t launch_seq = 0;       // waves launched so far
    uint64_t first_unchecked = 0;  // the first wave whose error record has not been read back
    uint64_t batch_tag = 0;        // tag of the current planning pass (one per collective and call of progress)
    uint64_t tag_counter = 0;      // tags handed out so far: later passes have larger tags, whether or not anything was launched in between
    std::vector<uint64_t> wave_tag;  // for the waves in flight (seq - first_unchecked): the tag of their planning pass
    hpl_stats_t stats{};
    int occ_reduce[2][2][3] = {};   // [bf16][fan][accumulator class]
    int occ_fanout = 0;
    struct Timed { cudaEvent_t a, b; int kind; };
    std::vector<Timed> timed;            // event pairs of launches not yet read back
    std::vector<cudaEvent_t> event_pool;
};

namespace hpl {

#ifdef HPL_DEBUG_BOUNDS
constexpr bool kDebugBounds = true;    // kernels look every buffer up in the directory and record accesses outside it
#else
constexpr bool kDebugBounds = false;
#endif

#define CUDA_TRY(x)                                  \
    do {                                             \
        if ((x) != cudaSuccess) return HPL_ERR_CUDA; \
    } while (0)

inline uint32_t elem_size(int dtype) { return dtype == HPL_BF16 ? 2u : 4u; }

inline uint32_t published_chunks(const hpl_ctx* c, const Object& o) {
    if (o.ready_bytes >= o.bytes) return o.C;
    return (uint32_t)(o.ready_bytes / c->cfg.chunk_bytes);
}

inline uint64_t object_elems(const Object& o) { return o.bytes / elem_size(o.dtype); }
inline uint64_t object_chunk_elems(const hpl_ctx* c, const Object& o) {
    return std::max<uint64_t>(1, std::min<uint64_t>(c->cfg.chunk_bytes, o.bytes) / elem_size(o.dtype));
}


// Operand i of an internal node u, in the association order of the tree: 0 = first child, 1 = the node's own
// object, i >= 2 = child i-1.  Returns the child's position, or -1 for the own object.
inline int operand_child(const ReduceTreeSchedule& s, int u, int i) { return i == 1 ? -1 : s.first_child(u) + (i == 0 ? 0 : i - 1); }
inline int operand_index_of_child(const ReduceTreeSchedule& s, int u, int child) {
    const int j = child - s.first_child(u);
    return j == 0 ? 0 : j + 1;
}

// directory.cpp
Object* find(hpl_ctx* c, int64_t id);
uint64_t logical_ready_elems(hpl_ctx* c, int64_t oid);
int64_t logical_delivered(hpl_ctx* c, int64_t oid);
int64_t logical_delivered_in(hpl_ctx* c, int64_t oid, const ReduceOp& op);
uint64_t produced_elems(hpl_ctx* c, const Object& o);
int alloc_row(hpl_ctx* c, Object& o);
int flush_directory(hpl_ctx* c);
int order_main_after_control(hpl_ctx* c);
int publish_counter(hpl_ctx* c, Object& o, uint32_t chunks, cudaStream_t s);
DeviceStatus* next_wave_status(hpl_ctx* c);
cudaEvent_t take_event(hpl_ctx* c);
void collect_kernel_times(hpl_ctx* c);
void release_object_memory(hpl_ctx* c, Object& o);
void* arena_alloc(hpl_ctx* c, uint64_t n, int home = -1);
hpl::Arena& arena_of_rank(hpl_ctx* c, int home);
void arena_release(hpl_ctx* c, void* p);
uint64_t check_guard(hpl_ctx* c, void* block);

// plan_reduce.cpp
int plan_reduce(hpl_ctx* c, ReduceOp& op, std::vector<PlannedReduceTask>& tasks);
int ensure_partial_buffer(hpl_ctx* c, ReduceOp& op, int pos, Object** out);
int launch_reduce_tasks(hpl_ctx* c, ReduceOp& op, std::vector<PlannedReduceTask>& tasks);
int launch_reduce_group(hpl_ctx* c, std::vector<std::pair<ReduceOp*, PlannedReduceTask*>>& group, bool bf16);
void apply_invalidation(hpl_ctx* c, ReduceOp& op, const ReduceInvalidation& inv);

// plan_bcast.cpp
int plan_bcast(hpl_ctx* c, BcastOp& op, std::vector<PlannedFanout>& tasks);
int launch_fanout_tasks(hpl_ctx* c, BcastOp& op, std::vector<PlannedFanout>& tasks);
int launch_fanout_group(hpl_ctx* c, std::vector<std::pair<BcastOp*, PlannedFanout>>& group);

// Brackets one launch with events when kernel timing is on (kind 0 = reduce, 1 = fan-out).
struct LaunchTimer {
    hpl_ctx* c;
    int kind;
    cudaEvent_t a = nullptr, b = nullptr;
    LaunchTimer(hpl_ctx* ctx, int k) : c(ctx), kind(k) {
        if (c->cfg.time_kernels) {
            a = take_event(c);
            b = take_event(c);
            if (a) cudaEventRecord(a, c->stream);
        }
    }
    ~LaunchTimer() {
        if (a && b) {
            cudaEventRecord(b, c->stream);
            c->timed.push_back({a, b, kind});
        }
    }
};

}  // namespace hpl
