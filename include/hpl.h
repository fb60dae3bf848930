/*
 * hpl -- chunk-pipelined reduce and broadcast over an object store, on one B200 (sm_100a).
 *
 * The calls follow the core interface of Hoplite (arXiv 2002.05814, Table 1: Get, Put, Delete,
 * Reduce) and its Section 3: objects are immutable buffers named by an id and owned by a task
 * worker; an object directory records, per object, its size and where copies are, each copy
 * with its progress (Section 3.2; the progress bit is refined here to a prefix counted in
 * chunks, Section 3.3); Reduce arranges whichever k of n source objects become ready first
 * into a degree-d tree filled in arrival order (Section 3.4.2); broadcast (many Gets of one
 * id, Section 3.4.1) forms a receiver-driven tree; a failed worker is taken out and the
 * schedules are re-formed (Section 3.5).  "Workers" are buffers in this GPU's memory and time
 * is a clock the caller sets (hpl_advance), so a schedule is a pure function of the timeline.
 *
 * Conventions
 *   - Every function returns HPL_OK (0) or a negative HPL_ERR_* code; nothing throws, nothing
 *     aborts.  hpl_strerror() names a code.
 *   - "device" pointers are addresses in the memory of the CUDA device that was current at
 *     hpl_init(); "host" pointers are ordinary process memory.
 *   - A context is not thread safe: one thread at a time.
 *   - Calls are events on the timeline and must come in non-decreasing time; events at the
 *     same time are to be issued failures first, then creations/puts, then reduce / broadcast /
 *     join requests (each group by ascending id).
 *   - All device work is enqueued on the stream given to hpl_init().  No call blocks on the
 *     device except hpl_get, hpl_get_host, hpl_sync and hpl_shutdown; every wait of a kernel on
 *     a progress counter is bounded by poll_budget_ns, after which the kernel gives up, records
 *     HPL_ERR_TIMEOUT and returns (the context stays usable).  One more wait exists: when the arena is full, a call
 *     that plans work waits for what is enqueued before it drops partial results (least recently used first; sources,
 *     Reduce outputs and store copies of host objects are never dropped) and, if need be, plans again.
 *
 * Capacities
 *   - The device directory has 4096 rows: one per published object (a put source, a joined receiver, a Reduce output,
 *     a partial result of a tree node).  A call that needs a row when none is free returns HPL_ERR_NOMEM and changes
 *     nothing; hpl_delete gives rows back.
 *   - A tree node has at most 638 children (the degree that counts is min(reduce_degree, k - 1); wider stars are
 *     refused with HPL_ERR_INVALID at hpl_reduce).  Objects, chunks and receivers per broadcast have no fixed limit:
 *     byte offsets and element counts are 64-bit, long receiver lists are served by several waves.
 */
#ifndef HPL_H_
#define HPL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HPL_OK                 0
#define HPL_ERR_INVALID       -1  /* bad argument: null, size 0, misaligned, unsupported dtype/op, time going back */
#define HPL_ERR_NOT_FOUND     -2  /* unknown object id */
#define HPL_ERR_EXISTS        -3  /* id already in use (objects are immutable, Section 2) */
#define HPL_ERR_TIMEOUT       -4  /* the object cannot be complete yet, or a bounded device wait expired */
#define HPL_ERR_INSUFFICIENT  -5  /* a Reduce is left with no live source */
#define HPL_ERR_FAILED_WORKER -6  /* the object's only copy was owned by a failed worker */
#define HPL_ERR_CUDA          -7  /* a CUDA call failed, or the context has no device (schedule-only) */
#define HPL_ERR_NOMEM         -8  /* the arena is exhausted.  From a call that plans work (hpl_progress, hpl_get, any event when
                                    eager): the collective that needed the room has nothing of that pass noted as done, what
                                    was planned before it runs, and the call may be repeated after room was made (hpl_delete) */

#define HPL_F32  0   /* 32-bit IEEE float */
#define HPL_BF16 1   /* bfloat16; reduced in fp32, result fp32 */

#define HPL_SUM 0
#define HPL_MIN 1    /* (b < a) ? b : a ; NaN inputs are outside the contract */
#define HPL_MAX 2    /* (a < b) ? b : a */

typedef struct hpl_ctx hpl_ctx;

typedef struct hpl_config {
    uint64_t chunk_bytes;     /* pipelining block (Section 3.3; 4 MB in the paper).  Multiple of 16.  An object
                                 smaller than this is one chunk. */
    int32_t  reduce_degree;   /* d of the reduce tree, >= 1 (Section 3.4.2, Eq. 1); 0 = chosen per Reduce among 1, 2 and
                                 k by Eq. 1 from model_latency_ns and model_bandwidth_bps (Section 4) */
    int32_t  bcast_degree;    /* concurrent sends per location, >= 1 (1 = the rule of Section 3.4.1) */
    uint64_t virt_chunk_ns;   /* virtual time for one chunk to cross one broadcast edge; 0 = chunk_bytes at 64 GiB/s */
    uint64_t poll_budget_ns;  /* bound on any device-side wait; 0 = 2 s */
    int32_t  eager;           /* 1: every event also plans and launches what has become runnable (as hpl_progress); an
                                 error of that planning is returned by the event's call, the event itself has been applied */
    int32_t  plan_ahead;      /* 1: chunks of a published object that are not ready yet are planned too; the
                                 kernels poll the directory's progress counters for them (bounded) */
    int32_t  fuse;            /* 1: a subtree whose inputs are all ready is reduced in registers in one pass
                                 (same association, same bits); 0: every tree node writes its partial result */
    int32_t  time_kernels;    /* 1: CUDA events are recorded around every kernel launch on the context's stream and
                                 summed into hpl_stats_t at the next wait (for benchmarks) */
    void*    arena;           /* device memory the library may use for the directory, partial results, reduce
                                 targets and copies of host objects; owned by the caller, must outlive the
                                 context.  NULL = schedule-only context: schedules are built and work is planned and counted
                                 (hpl_stats) exactly as with a device, but nothing is launched and hpl_get returns
                                 HPL_ERR_CUDA where it would otherwise succeed. */
    uint64_t arena_bytes;
    uint64_t model_latency_ns;     /* L of Eq. 1: latency of one hop; used only when reduce_degree == 0 */
    uint64_t model_bandwidth_bps;  /* B of Eq. 1: bytes per second into one node; used only when reduce_degree == 0 */
    int32_t  fuse_fanout;     /* 1: when the output of a Reduce is being broadcast (reduce followed by broadcast, the
                                 allreduce of Section 3.4.3), receivers that have joined take each result tile straight
                                 from the reduce pass -- the output is written once to the target and once to each of
                                 them and is not read again; 0: the broadcast always reads the target */
    int32_t  pipeline_chunks; /* worker-per-GPU mode: > 0 releases a task's chunk range in pieces of this many chunks, piece j
                                 one level after piece j-1, so that a tree level (or a broadcast hop) works on piece j
                                 while the next one works on piece j-1 -- Section 3.3's pipelining across the levels of a
                                 tree; 0: whole ranges, one level per tree level */
    uint64_t debug_guard_bytes;   /* testing aid, 0 = off: every block the library takes from the arena is followed by this
                                 many bytes of a canary pattern that no kernel may touch; checked when a block is
                                 released and by hpl_check_guards */
    int32_t  rank;            /* worker-per-GPU mode (below): this process' rank, 0 <= rank < world_size */
    int32_t  world_size;      /* 0 or 1: everything lives on this GPU.  > 1: see "Worker-per-GPU mode" */
} hpl_config;

/* Creates a context.  `cuda_stream` is a cudaStream_t (NULL = the legacy default stream).  Nothing is
 * allocated on the device: everything lives in cfg->arena.  Pinned host staging of a few KiB is allocated. */
int hpl_init(const hpl_config* cfg, void* cuda_stream, hpl_ctx** out);

/* Waits for enqueued work, releases host resources.  The arena and all object buffers stay the caller's. */
int hpl_shutdown(hpl_ctx* ctx);

/* Sets the clock for the events that follow (nanoseconds, non-decreasing).  Transfers of the virtual
 * broadcast model that land up to t_ns are applied first. */
int hpl_advance(hpl_ctx* ctx, uint64_t t_ns);

/* Declares a future: object `object_id`, owned by task worker `worker` (>= 0), `total_bytes` long
 * (a multiple of the element size).  Section 3.1: an ObjectID may be passed around before its value exists. */
int hpl_create(hpl_ctx* ctx, int64_t object_id, int32_t worker, uint64_t total_bytes, int32_t dtype);

/* Put (Table 1) with a DEVICE buffer, zero-copy.  `buf` points to the whole object (16-byte aligned); `bytes`
 * is the length of the prefix that is valid now.  The first call publishes the location as partial -- this is
 * the object's arrival (Section 3.2: the directory is told when Put is called, before the copy is done);
 * later calls extend the prefix (same `buf`, larger `bytes`); bytes == total marks it complete.  The store
 * borrows `buf`: the caller must not modify published bytes, nor free it before hpl_delete.  The bytes must
 * have been written by work enqueued earlier on the context's stream (or be visible before the call).
 * With plan_ahead = 1 the rule is stricter: the prefix must be VISIBLE AT THE CALL (written and waited for, or
 * produced on a stream the caller has synchronised).  The counter then goes out at once on a side stream, and a
 * polling wave that is already running on the context's stream consumes the bytes as soon as it sees it -- it
 * cannot be ordered behind producer work that sits after it on that stream. */
int hpl_put(hpl_ctx* ctx, int64_t object_id, const void* buf, uint64_t bytes);

/* Put (Table 1) with a HOST buffer: the store copies the prefix into its own device memory chunk by chunk,
 * asynchronously, publishing each chunk as it lands (Section 3.3: the copy into the store is pipelined with
 * the transfers that consume it).  `buf` must stay valid until hpl_sync/hpl_get returns; pinned memory makes
 * the copy overlap. */
int hpl_put_host(hpl_ctx* ctx, int64_t object_id, const void* buf, uint64_t bytes);

/* Many hpl_create / hpl_put / hpl_join calls at the current time, applied in array order exactly as the
 * single calls would be (so: ascending ids for equal-time events).  Stops at the first failure and returns
 * its code; *n_done (may be NULL) receives how many were applied.  They exist because a harness that stands
 * for many workers otherwise pays a foreign-call round trip per object. */
int hpl_create_batch(hpl_ctx* ctx, int32_t n, const int64_t* object_ids, const int32_t* workers, uint64_t total_bytes,
                     int32_t dtype, int32_t* n_done);
int hpl_put_batch(hpl_ctx* ctx, int32_t n, const int64_t* object_ids, const void* const* bufs /* host array of DEVICE
                  pointers */, const uint64_t* bytes, int32_t* n_done);
int hpl_join_batch(hpl_ctx* ctx, int32_t n, const int64_t* dst_ids, void* const* dst_bufs /* host array of DEVICE
                   pointers */, int32_t* n_done);

/* A timeline handed over in one call: `n` events in non-decreasing time, each applied exactly as the single call
 * of its kind would be (the same checks, the same codes).  A harness that stands for many task workers -- or a
 * framework that has collected a round's requests -- thereby pays one foreign call for a whole round instead of one
 * per worker.  Before each event the clock is set to its t_ns as by hpl_advance (t_ns == 0: the clock stays).
 * Stops at the first event that fails and returns its code; *n_done (may be NULL) receives how many were applied.
 * HPL_EV_GET writes its results back into the event (ptr, bytes): the array is in/out.
 *
 *   kind               fields used
 *   HPL_EV_CREATE      object_id, worker, bytes (total size), dtype            -> hpl_create
 *   HPL_EV_PUT         object_id, ptr (DEVICE buffer), bytes (valid prefix)     -> hpl_put
 *   HPL_EV_PUT_HOST    object_id, ptr (HOST buffer), bytes                      -> hpl_put_host
 *   HPL_EV_REDUCE      object_id (target), ids (host array of n_ids sources), k, op, dtype -> hpl_reduce
 *   HPL_EV_BROADCAST   object_id (source), ids (host array of n_ids receivers)  -> hpl_broadcast
 *   HPL_EV_JOIN        object_id (receiver), ptr (DEVICE buffer)                -> hpl_join
 *   HPL_EV_FAIL        worker                                                   -> hpl_fail
 *   HPL_EV_REJOIN      worker                                                   -> hpl_rejoin
 *   HPL_EV_PROGRESS    --                                                       -> hpl_progress
 *   HPL_EV_GET         object_id; out: ptr (device pointer), bytes              -> hpl_get
 *   HPL_EV_DELETE      object_id                                                -> hpl_delete
 *   HPL_EV_SYNC        --                                                       -> hpl_sync
 *   HPL_EV_MARK        ptr (a cudaEvent_t of the caller): recorded on the context's stream at this point of the
 *                      timeline, so that a harness can time parts of it on the device without leaving the call
 * Events at one time must come in the order the Conventions give (failures, creations / puts, requests). */
#define HPL_EV_CREATE    1
#define HPL_EV_PUT       2
#define HPL_EV_PUT_HOST  3
#define HPL_EV_REDUCE    4
#define HPL_EV_BROADCAST 5
#define HPL_EV_JOIN      6
#define HPL_EV_FAIL      7
#define HPL_EV_REJOIN    8
#define HPL_EV_PROGRESS  9
#define HPL_EV_GET       10
#define HPL_EV_DELETE    11
#define HPL_EV_SYNC      12
#define HPL_EV_MARK      13
typedef struct hpl_event {
    uint64_t t_ns;
    int32_t  kind;
    int32_t  worker;
    int64_t  object_id;
    void*    ptr;
    uint64_t bytes;
    const int64_t* ids;
    int32_t  n_ids;
    int32_t  k;
    int32_t  op;
    int32_t  dtype;
} hpl_event;
int hpl_submit(hpl_ctx* ctx, hpl_event* events, int32_t n, int32_t* n_done);

/* Many hpl_get calls, in array order; dev_ptrs[i] (may be NULL as a whole) receives the pointer of object i.
 * Stops at the first failure and returns its code. */
int hpl_get_batch(hpl_ctx* ctx, int32_t n, const int64_t* object_ids, const void** dev_ptrs, int32_t* n_done);

/* Reduce (Table 1, Section 3.4.2).  Non-blocking.  Creates `target_id` (fp32, library-owned, in the arena)
 * from `k_first_ready` of the `n` objects `src_ids` -- those that arrive first; ties by index in src_ids --
 * combined with `op` in the association order of the degree-d tree.  All sources have dtype `dtype` and one
 * size.  Sources may be futures. */
int hpl_reduce(hpl_ctx* ctx, int64_t target_id, const int64_t* src_ids, int32_t n, int32_t k_first_ready,
               int32_t op, int32_t dtype);

/* Registers `n` receiver copies `dst_ids` of object `src_id` (Section 3.4.1: a group of tasks that Get the
 * same object).  Each receiver was hpl_create'd with the source's size and dtype and is given its buffer by
 * hpl_join. */
int hpl_broadcast(hpl_ctx* ctx, int64_t src_id, const int64_t* dst_ids, int32_t n);

/* Receiver `dst_id` asks for the object now (its Get): the directory gives it one sender and lists it as a
 * partial copy.  `dst_buf`: device buffer of the object's size (16-byte aligned), caller-owned.  HPL_ERR_NOT_FOUND when
 * `dst_id` names no receiver of a broadcast (unknown, or an object that no hpl_broadcast listed). */
int hpl_join(hpl_ctx* ctx, int64_t dst_id, void* dst_buf);

/* Get (Table 1), read-only form (Section 3.3, immutable get): waits until the object is complete, returns a
 * device pointer into the store (valid until hpl_delete) and its size.  HPL_ERR_TIMEOUT if it cannot be
 * complete yet (state stays valid; retry after more events).  For a broadcast receiver the wait lets virtual
 * time run until its copy has landed. */
int hpl_get(hpl_ctx* ctx, int64_t object_id, const void** dev_ptr, uint64_t* bytes);

/* Get into HOST memory: as hpl_get, then copies the object to `dst` (capacity `cap` bytes) and waits. */
int hpl_get_host(hpl_ctx* ctx, int64_t object_id, void* dst, uint64_t cap);

/* Takes a task worker out (Section 3.5): every object and receiver copy it owns leaves all trees at once;
 * its buffers are never read by work enqueued after the call (what a broadcast copy of the worker can still serve
 * to receivers that have joined is copied by work the call itself enqueues first).  Reduce: the next ready source takes the
 * position, ancestors' partial results are cleared; with no spare left the tree shrinks.  Broadcast: the
 * receivers it was sending to ask again and resume from what they hold. */
int hpl_fail(hpl_ctx* ctx, int32_t worker);

/* The task framework has reconstructed failed worker `worker` (Section 3.5 lets a rebuilt task take part
 * again): the objects it owns are futures again -- not arrived, empty, to be Put again -- and the
 * receivers it owns may hpl_join again (a new location).  A Reduce counts a re-Put source as a new arrival:
 * it takes an open position or waits as a spare; a tree that shrank does not grow back.  A broadcast whose
 * SOURCE was lost is not revived.  Waits for enqueued work (directory rows are recycled). */
int hpl_rejoin(hpl_ctx* ctx, int32_t worker);

/* Eq. 1 / Section 4: the degree among 1, 2 and n with the smallest estimated reduce time
 * T(1) = n L + S/B, T(d) = L log_d n + d S/B (ties: the smaller degree).  Returns the degree (>= 1), or
 * HPL_ERR_INVALID.  Pure function: needs no context. */
int32_t hpl_choose_degree(int32_t n, uint64_t object_bytes, double latency_s, double bandwidth_bytes_per_s);

/* Delete (Table 1): drops the directory entry (and the collective it names, if it is a reduce target or a
 * broadcast source).  Library-owned memory returns to the arena; caller buffers may then be freed. */
int hpl_delete(hpl_ctx* ctx, int64_t object_id);

/* Plans and launches everything that is runnable now (non-blocking). */
int hpl_progress(hpl_ctx* ctx);

/* Waits for all launched work.  HPL_ERR_TIMEOUT if a device wait expired (the expired work is re-planned by
 * the next hpl_progress). */
int hpl_sync(hpl_ctx* ctx);

/* Serialises the schedule of the collective named by its reduce target id or broadcast source id (an id that is
 * both names the Reduce; any receiver id names the broadcast it belongs to) into
 * `words` (capacity `cap` 64-bit words); `*len` receives the number of words needed (HPL_ERR_INVALID if
 * cap is too small; *len is still set).
 *   Reduce:    0x48504C52, target, n, k requested, k now, d, #placements, {object, position}*, object at each
 *              position (-1 open), parent of each position, #spares, spares*, #edits, then per edit:
 *              epoch, kind (1 replaced by a spare, 2 position left open, 3 tree shrank), position, object
 *              that left, object now there, position it moved from, chunks the departed object had
 *              delivered, chunks the moved object had delivered, #cleared, cleared positions*.
 *   Broadcast: 0x48504C42, source, d, chunks, virtual chunk time, clock, #joined, then per receiver in join
 *              order: id, first sender, current sender (-1 none), first chunk fetched from it, join time,
 *              chunks held, alive, completion time (-1 not yet); #edits, then per edit: epoch, kind
 *              (1 new sender, 2 waits for a slot, 3 receiver left), receiver, old sender, new sender,
 *              chunks held, time. */
int hpl_schedule_dump(hpl_ctx* ctx, int64_t op_id, int64_t* words, uint64_t cap, uint64_t* len);

typedef struct hpl_stats_t {
    uint64_t kernel_launches;      /* kernels of this library launched so far */
    uint64_t reduce_tasks;         /* subtree tasks planned */
    uint64_t fanout_tasks;
    uint64_t tiles;                /* tiles planned (one CTA iteration each) */
    uint64_t bytes_read_planned;   /* bytes the planned tasks read */
    uint64_t bytes_written_planned;
    uint64_t device_timeouts;      /* bounded waits that expired */
    uint64_t arena_used;           /* bytes of the arena in use */
    uint64_t h2d_bytes;            /* copied by hpl_put_host */
    uint64_t d2h_bytes;            /* copied by hpl_get_host */
    uint64_t last_kernel_grid;     /* CTAs of the most recent launch */
    uint64_t reduce_launches;      /* launches of the reduce kernel */
    uint64_t fanout_launches;      /* launches of the fan-out kernel */
    uint64_t reduce_kernel_ns;     /* summed device time of reduce launches (time_kernels = 1; updated by waits) */
    uint64_t fanout_kernel_ns;
    uint64_t device_waits;         /* polls of a progress counter that did not succeed at the first look (updated by waits) */
    uint64_t fused_fanout_tasks;   /* reduce tasks that also wrote their result to broadcast receivers */
    uint64_t evictions;            /* partial results dropped, least recently used first, because the arena was full */
    uint64_t bounds_errors;        /* bounds-checking build of the library only: waves in which a tile lay outside its
                                      object (the tile is skipped and the wait reports HPL_ERR_TIMEOUT) */
} hpl_stats_t;

int hpl_stats(hpl_ctx* ctx, hpl_stats_t* out);

/* With debug_guard_bytes set: waits for the device, checks the canary behind every live arena block and returns in
 * *violations the number of canary bytes found changed so far (including those of blocks released earlier).
 * Without it: 0. */
int hpl_check_guards(hpl_ctx* ctx, uint64_t* violations);

const char* hpl_strerror(int code);

/* ---- Worker-per-GPU mode (world_size > 1): the paper's own setting -- one process and one GPU per node, objects live
 * where their worker runs, tree edges cross the interconnect (Sections 3.4 and 4; here NVLink peer memory).
 *
 * Every rank makes the SAME calls in the same order (the directory and the schedules are replicated; they are a pure
 * function of the timeline), and every rank executes only the tasks whose output lives on its GPU:
 *   - object `id` of worker w lives on rank w % world_size; a Reduce output lives on rank target_id % world_size; the
 *     partial result of a tree node lives with the node's object;
 *   - hpl_put / hpl_join take, on every rank, the address of the buffer IN THAT RANK'S address space: the owner its own
 *     allocation, the others a peer mapping of it (CUDA IPC; hpl_ipc_export / hpl_ipc_import);
 *   - every rank's arena has the same size and is peer-mapped by all others (hpl_set_peer_arena); allocation is
 *     replicated, so each rank knows where a remote partial result sits without asking;
 *   - a reduce task is run by the rank that owns its output and pulls remote operands over the link; a fan-out task is
 *     run by the rank that holds the copy being read and pushes to its receivers (one sender, at most d receivers:
 *     the tree edges of Section 3.4.1, followed strictly);
 *   - kernels never wait on another GPU.  Work is released in LEVELS: hpl_progress only plans; hpl_pending_levels
 *     says how many levels the plan has; hpl_run_level launches this rank's tasks of the next one.  Between two
 *     levels the caller waits for its own stream (hpl_sync) and runs a barrier over the live ranks.  When no level is
 *     left, hpl_progress is called again (receivers further down a broadcast tree are served by the next plan) until
 *     it plans nothing.  hpl_get does not drive this loop: it returns HPL_ERR_TIMEOUT until the object is done.
 *     While levels are pending, hpl_fail, hpl_rejoin, hpl_fail_rank and hpl_delete return HPL_ERR_INVALID: trees
 *     change and memory is recycled between plans, not inside one.  Bytes move only when the caller drives the levels:
 *     hpl_fail cannot first copy what a disappearing broadcast copy could still serve (as it does on one GPU), so a
 *     receiver that the schedule had given chunks which were never moved cannot complete from that copy afterwards
 *     -- drive the pending plan before taking a worker out.
 * plan_ahead, eager and hpl_put_host are not available in this mode (HPL_ERR_INVALID).  A rank that is lost is taken
 * out with hpl_fail_rank on every survivor: its workers fail (Section 3.5), and what lived on it is re-made
 * elsewhere; a Reduce whose output lived there is lost (HPL_ERR_FAILED_WORKER). */
int hpl_set_peer_arena(hpl_ctx* ctx, int32_t rank, void* arena_base /* DEVICE address, in this process, of that rank's arena */);
int hpl_pending_levels(hpl_ctx* ctx, int32_t* levels);
int hpl_run_level(hpl_ctx* ctx);
int hpl_fail_rank(hpl_ctx* ctx, int32_t rank);
/* Thin wrappers of CUDA IPC for the plumbing above.  Export: the 64-byte handle of the device ALLOCATION that holds
 * dev_ptr and the offset of dev_ptr inside it (a pointer handed out by a caching allocator need not be the start of
 * an allocation).  Import: maps another process' allocation and returns the address of the same byte in this
 * process.  Close: unmaps what hpl_ipc_import returned (before the owner frees the memory). */
int hpl_ipc_export(const void* dev_ptr, uint8_t handle[64], uint64_t* offset);
int hpl_ipc_import(const uint8_t handle[64], uint64_t offset, void** dev_ptr);
int hpl_ipc_close(void* dev_ptr);

/* Reduce for callers that cannot allocate device memory.  The paper has no counterpart: this is an
 * addition for users of this library who run where cudaMalloc is off limits -- allocator callbacks,
 * serving loops that have frozen their memory map, processes whose device memory all belongs to someone
 * else -- and who therefore cannot hand hpl_init an arena either.  It needs no context.
 *
 * Computes out[j] = op over the n objects src_bufs[0..n-1] (device pointers, 16-byte aligned, `elems`
 * elements of `dtype` each; the array src_bufs itself is host memory), all complete, taken as arriving in
 * index order, in the association order of the degree-`degree` tree -- the same bits hpl_reduce gives for
 * those arrivals.  `out`: device, fp32, `elems` elements, 16-byte aligned.  The work is enqueued on
 * `cuda_stream` and not waited for.
 *
 * The few KiB of device memory the kernel needs besides inputs and output (directory rows of the operands,
 * status record) are a fixed array inside the library image, held by every GPU that loads the library until
 * the process exits.  Hence the limits: n <= HPL_NOALLOC_MAX_SOURCES and elems <= HPL_NOALLOC_MAX_ELEMS;
 * a tree deeper than the kernel can fuse in registers (8 accumulators) would be refused too (no degree reaches
 * that depth within the limit on n).  Anything beyond
 * returns HPL_ERR_INVALID and does nothing.  No cudaMalloc / cudaFree / allocating routine is called.
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress) and the SM count;
 * make that first call outside any stream capture.  All calls share the one array and each call rewrites
 * it: two calls whose kernels may overlap on the GPU (different streams, no ordering) race -- order them. */
#define HPL_NOALLOC_MAX_SOURCES 256
#define HPL_NOALLOC_MAX_ELEMS   (1ull << 32)
int hpl_reduce_noalloc(const void* const* src_bufs, int32_t n, int32_t degree, int32_t op, int32_t dtype,
                       uint64_t elems, void* out, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* HPL_H_ */
