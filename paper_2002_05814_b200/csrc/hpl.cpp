// Host side of the library: object directory, event handling, planners that turn the current
// schedules into waves of kernel tasks, and the C ABI (include/hpl.h).
//
// Division of labour (arXiv 2002.05814, Section 3): the schedule builders (sched_reduce.*,
// sched_bcast.*) decide WHO combines / forwards WHAT, as a function of the event timeline only.
// The planners below decide HOW the pending part of those schedules is executed on the GPU right
// now: which subtrees of a reduce tree are complete for which chunks (those are fused into one
// pass in registers), which partial results must be materialised, which receivers can be served
// from which copy.  Execution order is free as long as the association order of the tree is
// kept, so the bits do not depend on it.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstddef>
#include <cstdlib>
#include <cstring>
#include <map>
#include <memory>
#include <unordered_map>
#include <vector>

#include "../../include/hpl.h"
#include "device_types.h"
#include "sched_bcast.h"
#include "sched_reduce.h"

using namespace hpl;

namespace {

constexpr uint32_t kMaxRows = 4096;
constexpr uint32_t kStatusSlots = 256;   // one error record per wave in flight; beyond that the last one is shared
constexpr uint32_t kMaxChunks = 1u << 20;
constexpr uint64_t kAlign = 256;

// ------------------------------------------------------------------------------------------ small utilities
struct IntervalSet {  // disjoint, sorted [a, b) chunk ranges
    std::vector<std::pair<uint32_t, uint32_t>> iv;
    void clear() { iv.clear(); }
    bool contains(uint32_t a, uint32_t b) const {
        for (auto& x : iv)
            if (x.first <= a && b <= x.second) return true;
        return false;
    }
    void add(uint32_t a, uint32_t b) {
        if (a >= b) return;
        std::vector<std::pair<uint32_t, uint32_t>> out;
        for (auto& x : iv) {
            if (x.second < a || b < x.first)
                out.push_back(x);
            else {
                a = std::min(a, x.first);
                b = std::max(b, x.second);
            }
        }
        out.emplace_back(a, b);
        std::sort(out.begin(), out.end());
        iv.swap(out);
    }
    void remove(uint32_t a, uint32_t b) {
        std::vector<std::pair<uint32_t, uint32_t>> out;
        for (auto& x : iv) {
            if (x.second <= a || b <= x.first) {
                out.push_back(x);
                continue;
            }
            if (x.first < a) out.emplace_back(x.first, a);
            if (b < x.second) out.emplace_back(b, x.second);
        }
        iv.swap(out);
    }
    void breakpoints(std::vector<uint32_t>& bp) const {
        for (auto& x : iv) {
            bp.push_back(x.first);
            bp.push_back(x.second);
        }
    }
};

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
};

struct Journal {  // what was planned since the last successful wait (undone if a device wait expires)
    // tag: number of waves launched before the planning pass that made the entry (its waves have seq >= tag)
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
};

struct BcastOp {
    int64_t src;
    std::unique_ptr<BroadcastTreeSchedule> sched;
    std::vector<int64_t> dsts;
    std::vector<int64_t> phys_have;  // per location index: chunks physically planned (index 0 unused)
    uint64_t seq;
};

}  // namespace

struct hpl_ctx {
    hpl_config cfg{};
    cudaStream_t stream = nullptr, copy_stream = nullptr, ctl_stream = nullptr;
    cudaEvent_t copy_ev = nullptr, ctl_ev = nullptr;
    bool device = false;
    bool copy_pending = false;
    bool ctl_pending = false;   // directory updates on the control stream not yet ordered before the main stream
    int n_sm = 0;
    uint64_t now = 0, tau = 1, seq = 0;
    int64_t next_internal = -1;  // ids of partial buffers: negative, never visible outside
    Arena arena;
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
    Journal journal;
    bool work_in_flight = false;
    uint64_t launch_seq = 0;       // waves launched so far
    uint64_t first_unchecked = 0;  // the first wave whose error record has not been read back
    uint64_t batch_tag = 0;        // launch_seq when the current planning pass began
    std::vector<uint64_t> wave_tag;  // for the waves in flight (seq - first_unchecked): the tag of their planning pass
    hpl_stats_t stats{};
    int occ_reduce[2][3] = {{0, 0, 0}, {0, 0, 0}};
    int occ_fanout = 0;
    struct Timed { cudaEvent_t a, b; int kind; };
    std::vector<Timed> timed;            // event pairs of launches not yet read back
    std::vector<cudaEvent_t> event_pool;
};

namespace {

inline uint32_t elem_size(int dtype) { return dtype == HPL_BF16 ? 2u : 4u; }

inline uint32_t published_chunks(const hpl_ctx* c, const Object& o) {
    if (o.ready_bytes >= o.bytes) return o.C;
    return (uint32_t)(o.ready_bytes / c->cfg.chunk_bytes);
}

Object* find(hpl_ctx* c, int64_t id) {
    auto it = c->objects.find(id);
    return it == c->objects.end() ? nullptr : &it->second;
}

inline uint64_t object_elems(const Object& o) { return o.bytes / elem_size(o.dtype); }
inline uint64_t object_chunk_elems(const hpl_ctx* c, const Object& o) {
    return std::max<uint64_t>(1, std::min<uint64_t>(c->cfg.chunk_bytes, o.bytes) / elem_size(o.dtype));
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

#define CUDA_TRY(x)                                  \
    do {                                             \
        if ((x) != cudaSuccess) return HPL_ERR_CUDA; \
    } while (0)

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
    // With plan-ahead a kernel that polls may occupy the main stream for a while, so directory rows travel
    // on the control stream (tiny copies only) and the main stream is ordered after it before each launch.
    if (!c->device) {
        // schedule-only context: the mirror is all there is (the planners run, nothing is launched)
    } else if (c->cfg.plan_ahead) {
        CUDA_TRY(cudaMemcpyAsync(c->d_dir + o.row, &r, sizeof(DirRow), cudaMemcpyHostToDevice, c->ctl_stream));
        c->ctl_pending = true;
    } else {
        c->dirty_rows.push_back(o.row);   // travels with the next flush, before the next launch
    }
    return HPL_OK;
}

constexpr uint32_t kStageRows = 4 * kMaxRows;

// Batched mode (no plan-ahead): all rows changed since the last flush go to the device in one copy per run of
// consecutive rows, from an immutable pinned snapshot, ordered on the main stream before whatever is
// launched next.  A Put is then a few stores on the host; its cost on the device is amortised over the batch.
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
            CUDA_TRY(cudaStreamSynchronize(c->stream));   // every earlier snapshot has been consumed
            c->stage_cursor = 0;
        }
        DirRow* snap = c->h_stage + c->stage_cursor;
        std::memcpy(snap, c->h_dir + c->dirty_rows[i], n * sizeof(DirRow));
        CUDA_TRY(cudaMemcpyAsync(c->d_dir + c->dirty_rows[i], snap, n * sizeof(DirRow), cudaMemcpyHostToDevice, c->stream));
        c->stage_cursor += n;
        i = j;
    }
    c->dirty_rows.clear();
    return HPL_OK;
}

int order_main_after_control(hpl_ctx* c) {
    if (!c->ctl_pending) return HPL_OK;
    CUDA_TRY(cudaEventRecord(c->ctl_ev, c->ctl_stream));
    CUDA_TRY(cudaStreamWaitEvent(c->stream, c->ctl_ev, 0));
    c->ctl_pending = false;
    return HPL_OK;
}

// Publishes the chunk prefix of a put object in the device directory, ordered on `s`.
int publish_counter(hpl_ctx* c, Object& o, uint32_t chunks, cudaStream_t s) {
    if (o.row < 0) return HPL_OK;
    c->h_dir[o.row].ready_chunks = chunks;   // the host mirror always holds the published value
    if (!c->device) return HPL_OK;
    if (s == c->stream && !c->cfg.plan_ahead) {
        c->dirty_rows.push_back(o.row);
        return HPL_OK;
    }
    CUDA_TRY(cudaMemcpyAsync(&c->d_dir[o.row].ready_chunks, &c->h_iota[chunks], sizeof(uint32_t), cudaMemcpyHostToDevice, s));
    return HPL_OK;
}

int sync_and_check(hpl_ctx* c);
int progress(hpl_ctx* c);

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

void release_object_memory(hpl_ctx* c, Object& o) {
    if (o.lib_owned && o.ptr) c->arena.release(o.ptr);
    o.ptr = nullptr;
    if (o.row >= 0) c->free_rows.push_back(o.row);
    o.row = -1;
}

// ------------------------------------------------------------------------------------------ reduce planner
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
        return HPL_OK;
    }
    Object o;
    o.id = c->next_internal--;
    o.kind = OBJ_PARTIAL;
    o.bytes = op.elems * 4;
    o.dtype = HPL_F32;
    o.C = op.C;
    o.lib_owned = true;
    o.seq = c->seq++;
    o.ptr = c->arena.alloc(o.bytes);
    if (!o.ptr) return HPL_ERR_NOMEM;
    o.ready_bytes = o.bytes;
    int rc = alloc_row(c, o);
    if (rc != HPL_OK) {
        c->arena.release(o.ptr);
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
        st.row = (uint32_t)find(p.c, q == 0 ? op.target : op.partial_key[q])->row;
    } else {
        st.kind = op.in_dtype == HPL_BF16 ? SRC_BF16 : SRC_F32;
        st.row = (uint32_t)find(p.c, op.sched->object_at(q))->row;
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

// Operand i of an internal node u, in the association order of the tree: 0 = first child, 1 = the node's own
// object, i >= 2 = child i-1.  Returns the child's position, or -1 for the own object.
inline int operand_child(const ReduceTreeSchedule& s, int u, int i) { return i == 1 ? -1 : s.first_child(u) + (i == 0 ? 0 : i - 1); }
inline int operand_index_of_child(const ReduceTreeSchedule& s, int u, int child) {
    const int j = child - s.first_child(u);
    return j == 0 ? 0 : j + 1;
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

int plan_reduce(hpl_ctx* c, ReduceOp& op, std::vector<PlannedReduceTask>& tasks) {
    ReduceTreeSchedule& s = *op.sched;
    const int k = s.k();
    if (k <= 0) return HPL_OK;
    std::vector<uint32_t> ready(k, 0), landed(k, 0);
    std::vector<uint32_t> bp = {0u, op.C};
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
        ReducePlanCtx p;
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
    return HPL_OK;
}

int occ_index(int n_acc) { return n_acc <= 2 ? 0 : (n_acc <= 4 ? 1 : 2); }

int launch_reduce_tasks(hpl_ctx* c, ReduceOp& op, std::vector<PlannedReduceTask>& tasks) {
    if (tasks.empty()) return HPL_OK;
    int max_level = 0;
    for (auto& t : tasks) max_level = std::max(max_level, t.level);
    const bool bf16 = op.in_dtype == HPL_BF16;
    const uint32_t tpc_full = (op.chunk_elems + kTileElems - 1) / kTileElems;
    for (int level = 1; level <= max_level; ++level) {
        size_t i = 0;
        std::vector<PlannedReduceTask*> lv;
        for (auto& t : tasks)
            if (t.level == level) lv.push_back(&t);
        while (i < lv.size()) {
            static thread_local ReduceWave w;
            w.dir = c->d_dir;
            w.status = nullptr;
            w.budget_ns = c->cfg.poll_budget_ns;
            w.n_tasks = 0;
            w.total_tiles = 0;
            uint32_t n_steps = 0;
            int n_acc = 1;
            while (i < lv.size() && w.n_tasks < (uint32_t)kMaxTasksPerWave &&
                   n_steps + lv[i]->steps.size() <= (size_t)kMaxStepsPerWave) {
                PlannedReduceTask& t = *lv[i];
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
                d.pad = 0;
                std::memcpy(&w.steps[n_steps], t.steps.data(), t.steps.size() * sizeof(ReduceStep));
                n_steps += d.n_steps;
                w.total_tiles += (t.b - t.a) * tpc_full;
                n_acc = std::max(n_acc, t.n_acc);
                // accounting: bytes the task moves
                uint64_t e_lo = (uint64_t)t.a * op.chunk_elems, e_hi = std::min<uint64_t>((uint64_t)t.b * op.chunk_elems, op.elems);
                for (auto& st : t.steps)
                    if (st.code != OPC_ADD_ACC) c->stats.bytes_read_planned += (e_hi - e_lo) * (st.kind == SRC_BF16 ? 2 : 4);
                c->stats.bytes_written_planned += (e_hi - e_lo) * 4;
                c->stats.reduce_tasks++;
                ++i;
            }
            if (w.n_tasks == 0) return HPL_ERR_INVALID;  // a single task larger than a wave: tree too wide
            if (!c->device) {   // schedule-only context: the wave is planned and counted, not run
                c->stats.kernel_launches++;
                c->stats.reduce_launches++;
                c->stats.tiles += w.total_tiles;
                continue;
            }
            int& occ = c->occ_reduce[bf16 ? 1 : 0][occ_index(n_acc)];
            if (occ == 0) occ = reduce_ctas_per_sm(n_acc, bf16);
            int grid = (int)std::min<uint64_t>(w.total_tiles, (uint64_t)c->n_sm * occ);
            if (grid < 1) grid = 1;
            if (flush_directory(c) != HPL_OK) return HPL_ERR_CUDA;   // rows of partial results created while planning
            w.status = next_wave_status(c);
            {
                LaunchTimer timer(c, 0);
                if (launch_reduce_wave(w, n_acc, bf16, grid, c->stream) != 0) return HPL_ERR_CUDA;
            }
            c->stats.kernel_launches++;
            c->stats.reduce_launches++;
            c->stats.tiles += w.total_tiles;
            c->stats.last_kernel_grid = (uint64_t)grid;
            c->work_in_flight = true;
        }
    }
    return HPL_OK;
}

// ------------------------------------------------------------------------------------------ broadcast planner
struct PlannedFanout {
    int loc;  // location index read from
    uint32_t a, b;
    bool poll;
    std::vector<int> dst;  // location indices written
};

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
        std::map<int, std::vector<int>> groups;  // read location -> receivers
        for (int r = 1; r < (int)locs.size(); ++r) {
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
            const bool poll = (g.first == 0) && (src_landed < b);
            bool merged = false;
            for (auto& prev : tasks) {
                if (prev.loc == g.first && prev.b == a && prev.poll == poll && prev.dst == g.second) {
                    prev.b = b;
                    merged = true;
                    break;
                }
            }
            if (!merged) tasks.push_back(PlannedFanout{g.first, a, b, poll, g.second});
        }
    }
    return HPL_OK;
}

int launch_fanout_tasks(hpl_ctx* c, BcastOp& op, std::vector<PlannedFanout>& tasks) {
    if (tasks.empty()) return HPL_OK;
    Object* src = find(c, op.src);
    const auto& locs = op.sched->locations();
    const uint64_t chunk_bytes = c->cfg.chunk_bytes;
    const uint32_t tpc = (uint32_t)((std::min<uint64_t>(chunk_bytes, src->bytes) + kFanoutTileBytes - 1) / kFanoutTileBytes);
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
            PlannedFanout& t = tasks[i];
            if (t.dst.size() > (size_t)kMaxFanoutDst) {
                // more receivers than one task holds: split the receiver list
                PlannedFanout rest = t;
                rest.dst.assign(t.dst.begin() + kMaxFanoutDst, t.dst.end());
                t.dst.resize(kMaxFanoutDst);
                tasks.insert(tasks.begin() + i + 1, rest);
                continue;
            }
            if (n_dst + tasks[i].dst.size() > (size_t)kMaxFanoutDst) break;
            PlannedFanout& tt = tasks[i];
            FanoutTask& d = w.tasks[w.n_tasks++];
            Object* lo = tt.loc == 0 ? src : find(c, locs[tt.loc].obj);
            d.src_row = (uint32_t)lo->row;
            d.c_begin = tt.a;
            d.c_end = tt.b;
            d.tiles_per_chunk = tpc;
            d.tile_begin = w.total_tiles;
            d.dst_begin = n_dst;
            d.n_dst = (uint32_t)tt.dst.size();
            d.poll = tt.poll ? 1u : 0u;
            d.bytes = src->bytes;
            d.chunk_bytes = chunk_bytes;
            for (int r : tt.dst) w.dst_rows[n_dst++] = (uint32_t)find(c, locs[r].obj)->row;
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
        int grid = (int)std::min<uint64_t>(w.total_tiles, (uint64_t)c->n_sm * c->occ_fanout);
        if (grid < 1) grid = 1;
        if (flush_directory(c) != HPL_OK) return HPL_ERR_CUDA;
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

// ------------------------------------------------------------------------------------------ progress / sync
int progress(hpl_ctx* c) {
    // (a schedule-only context plans as well -- its planned tasks are counted, nothing is launched)
    {
        int rc = order_main_after_control(c);
        if (rc != HPL_OK) return rc;
        rc = flush_directory(c);
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
    // collectives in creation order, so that one that consumes another's output (composed Reduce, reduce
    // followed by broadcast) is planned after its producer and launched behind it on the stream
    auto ri = c->reduces.begin();
    auto bi = c->bcasts.begin();
    while (ri != c->reduces.end() || bi != c->bcasts.end()) {
        const bool take_reduce = bi == c->bcasts.end() || (ri != c->reduces.end() && ri->first < bi->first);
        c->batch_tag = c->launch_seq;
        if (take_reduce) {
            std::vector<PlannedReduceTask> tasks;
            int rc = plan_reduce(c, ri->second, tasks);
            if (rc != HPL_OK) return rc;
            rc = launch_reduce_tasks(c, ri->second, tasks);
            if (rc != HPL_OK) return rc;
            ++ri;
        } else {
            std::vector<PlannedFanout> tasks;
            int rc = plan_bcast(c, bi->second, tasks);
            if (rc != HPL_OK) return rc;
            rc = launch_fanout_tasks(c, bi->second, tasks);
            if (rc != HPL_OK) return rc;
            ++bi;
        }
    }
    return HPL_OK;
}

// Voids what was planned by the passes whose waves have seq >= from_tag (a wave of that pass gave up, and
// later passes may have built on it); earlier passes ran to completion and are kept.
void undo_journal(hpl_ctx* c, uint64_t from_tag) {
    for (auto& e : c->journal.r) {
        if (e.tag < from_tag) continue;
        auto it = c->reduce_of_target.find(e.target);
        if (it == c->reduce_of_target.end()) continue;
        ReduceOp& op = c->reduces.at(it->second);
        // back to nothing, not to the earlier value: a task that gave up half way may have updated part of the
        // buffer in place, so what it held before is gone as well
        if (e.pos < (int)op.merged.size()) op.merged[e.pos].set(e.a, e.b, 0);
    }
    for (auto it = c->journal.b.rbegin(); it != c->journal.b.rend(); ++it) {
        if (it->tag < from_tag) continue;
        auto f = c->bcast_of_src.find(it->src);
        if (f == c->bcast_of_src.end()) continue;
        BcastOp& op = c->bcasts.at(f->second);
        if (it->loc < (int)op.phys_have.size()) op.phys_have[it->loc] = it->old_have;
    }
    c->journal.clear();
}

int sync_and_check(hpl_ctx* c) {
    if (!c->device) {
        c->journal.clear();
        return HPL_OK;
    }
    if (c->copy_pending || c->ctl_pending) {
        CUDA_TRY(cudaStreamSynchronize(c->ctl_stream));
        CUDA_TRY(cudaStreamSynchronize(c->copy_stream));
        c->copy_pending = false;
        c->ctl_pending = false;
        for (auto& kv : c->objects)
            if (kv.second.async_counter) kv.second.landed = published_chunks(c, kv.second);
    }
    if (!c->work_in_flight) {   // nothing of the library's is running: nothing to wait for
        c->journal.clear();
        return HPL_OK;
    }
    const uint32_t used = (uint32_t)std::min<uint64_t>(c->launch_seq - c->first_unchecked, kStatusSlots);
    CUDA_TRY(cudaMemcpyAsync(c->h_status, c->d_status, sizeof(DeviceStatus) * used, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(cudaStreamSynchronize(c->stream));
    c->work_in_flight = false;
    collect_kernel_times(c);
    bool failed = false;
    uint64_t from_tag = ~0ull;
    for (uint32_t i = 0; i < used; ++i) {
        c->stats.device_waits += c->h_status[i].waits;
        if (!c->h_status[i].error) continue;
        failed = true;
        // the record in the last slot may stand for several waves: the earliest of them decides
        const uint64_t tag = c->wave_tag[i];
        from_tag = std::min(from_tag, tag);
    }
    c->first_unchecked = c->launch_seq;
    c->wave_tag.clear();
    // the records are cleared behind everything launched so far; later launches are ordered after that
    CUDA_TRY(cudaMemsetAsync(c->d_status, 0, sizeof(DeviceStatus) * used, c->stream));
    if (failed) {
        c->stats.device_timeouts++;
        undo_journal(c, from_tag);
        return HPL_ERR_TIMEOUT;
    }
    c->journal.clear();
    return HPL_OK;
}

int after_event(hpl_ctx* c) { return c->cfg.eager ? progress(c) : HPL_OK; }

// After every event: a broadcast whose source is a Reduce output learns how far that output has got.
void refresh_composed(hpl_ctx* c) {
    for (auto& kv : c->bcasts) {
        Object* src = find(c, kv.second.src);
        if (src && src->kind == OBJ_TARGET) kv.second.sched->source_progress((int64_t)c->now, logical_delivered(c, src->id));
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

// A position's own object changed, or the position disappeared: its buffer is void, and so is, in every
// ancestor, whatever was merged from the child on that path onwards.  What an ancestor had merged BEFORE that
// child (its earlier operands) is untouched and kept -- healthy chunks are not redone.
void apply_invalidation(ReduceOp& op, const ReduceInvalidation& inv) {
    const int k = op.sched->k();
    ReduceTreeSchedule& s = *op.sched;
    if (inv.shrank) {
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

void notify_arrival(hpl_ctx* c, Object& o) {
    for (auto& kv : c->reduces)
        if (kv.second.sched->has_source(o.id)) kv.second.sched->arrive(o.id);
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
    hpl_ctx* c = new (std::nothrow) hpl_ctx();
    if (!c) return HPL_ERR_NOMEM;
    c->cfg = *cfg;
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
            c->ctl_pending = true;
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
    const bool first = !o->arrived;
    if (!first && !o->from_host) return HPL_ERR_INVALID;
    if (first) {
        o->ptr = c->arena.alloc(o->bytes);
        if (!o->ptr) return HPL_ERR_NOMEM;
        o->lib_owned = true;
        o->from_host = true;
        o->async_counter = true;
        rc = alloc_row(c, *o);
        if (rc != HPL_OK) {
            c->arena.release(o->ptr);
            o->ptr = nullptr;
            o->lib_owned = false;
            return rc;
        }
        // the row (pointer) must be in the directory before any copy-stream counter update can matter
        cudaStream_t row_stream = c->cfg.plan_ahead ? c->ctl_stream : c->stream;
        rc = flush_directory(c);
        if (rc != HPL_OK) return rc;
        CUDA_TRY(cudaEventRecord(c->copy_ev, row_stream));
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
    for (int64_t s : srcs) {
        Object* o = find(c, s);
        if (!o) return HPL_ERR_NOT_FOUND;
        if (o->dtype != dtype || (bytes && o->bytes != bytes) || o->kind == OBJ_RECEIVER) return HPL_ERR_INVALID;
        bytes = o->bytes;
        if (o->alive) ++live;
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
        t.ptr = c->arena.alloc(t.bytes);
        if (!t.ptr) return HPL_ERR_NOMEM;
        int rc = alloc_row(c, t);
        if (rc != HPL_OK) {
            c->arena.release(t.ptr);
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
        if (t.ptr) c->arena.release(t.ptr);
        if (t.row >= 0) c->free_rows.push_back(t.row);
        c->objects.erase(target);
        return HPL_ERR_INVALID;
    }
    r.sched.reset(new ReduceTreeSchedule(srcs, k, degree));
    r.red_op = op;
    r.in_dtype = dtype;
    r.elems = elems;
    r.C = find(c, srcs[0])->C;          // chunks of this Reduce follow its inputs (chunk_bytes of the input dtype)
    r.chunk_elems = (uint32_t)(std::min<uint64_t>(c->cfg.chunk_bytes, bytes) / elem_size(dtype));
    if (r.chunk_elems == 0) r.chunk_elems = 1;
    r.seq = c->seq++;
    ReduceOp* rp = &r;
    auto dl = [c, rp](int64_t o) { return logical_delivered_in(c, o, *rp); };
    for (int64_t s : srcs)
        if (!find(c, s)->alive) r.sched->fail(s, 0, dl);  // sources lost before the call never take part
    std::vector<std::pair<std::pair<int64_t, int>, int64_t>> arrived;
    for (int i = 0; i < n; ++i) {
        Object* o = find(c, srcs[i]);
        if (o->alive && o->arrived) arrived.push_back({{o->t_arrival, i}, o->id});
    }
    std::sort(arrived.begin(), arrived.end());
    for (auto& a : arrived) r.sched->arrive(a.second);
    r.merged.assign(r.sched->k(), IntervalMap());
    r.partial_key.assign(r.sched->k(), 0);
    const uint64_t key = r.seq;
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
        d->ready_bytes = 0;
        int rc = alloc_row(c, *d);
        if (rc != HPL_OK) return rc;
    }
    b.sched->join((int64_t)c->now, dst_id);
    return after_event(c);
}

int hpl_fail(hpl_ctx* c, int32_t worker) {
    if (!c || worker < 0) return HPL_ERR_INVALID;
    std::vector<Object*> lost;
    for (auto& kv : c->objects)
        if (kv.second.worker == worker && kv.second.alive) lost.push_back(&kv.second);
    std::sort(lost.begin(), lost.end(), [](Object* a, Object* b) { return a->seq < b->seq; });
    for (Object* o : lost) o->alive = false;
    for (auto& kv : c->reduces) {
        ReduceOp& op = kv.second;
        ReduceOp* rp = &op;
        auto dl = [c, rp](int64_t o) { return logical_delivered_in(c, o, *rp); };
        for (Object* o : lost) {
            if (!op.sched->has_source(o->id)) continue;
            ReduceInvalidation inv = op.sched->fail(o->id, logical_delivered_in(c, o->id, op), dl);
            apply_invalidation(op, inv);
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
        for (auto& rk : c->reduces)
            if (rk.second.sched->has_source(o.id)) rk.second.sched->rejoin(o.id);
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
        int rc = progress(c);   // whatever can run now runs, even if the target cannot complete yet
        if (rc != HPL_OK) return rc;
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
        if (li < 0) return HPL_ERR_TIMEOUT;  // never joined
        if (li >= (int)op.phys_have.size() || op.phys_have[li] < (int64_t)o->C) {
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
        if (!c->device) return HPL_ERR_CUDA;
        if (li < (int)op.phys_have.size() && op.phys_have[li] >= (int64_t)o->C && !c->work_in_flight && !c->copy_pending) {
            if (dev_ptr) *dev_ptr = o->ptr;   // already copied and waited for
            if (bytes) *bytes = o->bytes;
            return HPL_OK;
        }
        int rc = progress(c);
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
    if (o->kind == OBJ_RECEIVER) return HPL_ERR_INVALID;  // deleted with its broadcast
    for (auto& kv : c->reduces)
        if (kv.second.sched->has_source(id)) return HPL_ERR_INVALID;  // still referenced by a Reduce
    if (c->device) {
        // rows and arena memory are recycled only when nothing enqueued can still read them
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
    else
        return HPL_ERR_NOT_FOUND;
    *len = w.size();
    if (!words || cap < w.size()) return HPL_ERR_INVALID;
    std::memcpy(words, w.data(), w.size() * sizeof(int64_t));
    return HPL_OK;
}

int hpl_stats(hpl_ctx* c, hpl_stats_t* out) {
    if (!c || !out) return HPL_ERR_INVALID;
    c->stats.arena_used = c->arena.used;
    *out = c->stats;
    return HPL_OK;
}

}  // extern "C"
