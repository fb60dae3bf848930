// sm_100a kernels of the reduce / broadcast hot path.
//
//  reduce_wave_kernel  -- persistent grid over the tiles of a wave of subtree tasks.  A task is a
//      fused evaluation of a subtree of the reduce tree (arXiv 2002.05814, Section 3.4.2) over a
//      range of chunks: a short program of LOAD / ADD_LOAD / ADD_ACC steps, executed per tile with
//      the accumulators in registers, in exactly the association order of the tree, fp32, no
//      contraction, no fast-math.  Before a chunk is touched the progress counters of its operands
//      are polled in the device directory (bounded wait), which is how a chunk that is still being
//      copied into the store is consumed as soon as it lands (Section 3.3).
//  fanout_wave_kernel  -- reads each tile of a chunk once into shared memory and writes it to every
//      receiver of the task with bulk copies (Section 3.4.1: the receivers of one sender subtree), same polling.
//
// Global reads are 16 bytes per thread, coalesced and L2-only (.cg) because every byte is used once.
// The reduce kernel stages its operand tiles through shared memory with cp.async, several steps ahead
// of the adds, so that 80 KiB and more per SM are in flight without holding registers.
#include <cuda_runtime.h>

#include <array>
#include <mutex>
#include <vector>

#include "device_types.h"

namespace hpl {

__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ unsigned int load_acquire_sys(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Waits until dir[row].ready_chunks > chunk.  Bounded twice: by the wave's time budget measured from
// the kernel's start and by an iteration cap.  On expiry records the wait in *status and returns false.
__device__ bool wait_chunk(const DirRow* dir, DeviceStatus* status, unsigned int row, unsigned int chunk,
                           unsigned long long t_start, unsigned long long budget_ns) {
    const unsigned int* flag = &dir[row].ready_chunks;
    if (load_acquire_sys(flag) > chunk) return true;
    atomicAdd(&status->waits, 1ull);
    const unsigned long long max_iter = budget_ns / 128ull + 1024ull;
    for (unsigned long long it = 0; it < max_iter; ++it) {
        __nanosleep(200);
        if (load_acquire_sys(flag) > chunk) return true;
        if (*reinterpret_cast<volatile unsigned int*>(&status->abort)) return false;
        if (global_timer_ns() - t_start > budget_ns) break;
    }
    if (atomicCAS(&status->error, 0u, 1u) == 0u) {
        status->row = row;
        status->chunk = chunk;
    }
    __threadfence();
    *reinterpret_cast<volatile unsigned int*>(&status->abort) = 1u;
    return false;
}

#ifdef HPL_DEBUG_BOUNDS
// Bounds-checking build: every buffer a tile touches is looked up in the device directory; the address the wave
// carries must be the row's, and the bytes touched must lie inside the object.  A violation is recorded (error 2)
// and the tile is skipped instead of being accessed.
__device__ bool range_ok(const DirRow* dir, DeviceStatus* status, unsigned int row, unsigned long long ptr, unsigned long long lo,
                         unsigned long long hi, unsigned int chunk) {
    const DirRow r = dir[row];
    if ((r.ptr & ((1ull << kRecShift) - 1)) == (ptr & ((1ull << kRecShift) - 1)) && lo <= hi && hi <= r.bytes) return true;
    if (atomicCAS(&status->error, 0u, 2u) == 0u) {
        status->row = row;
        status->chunk = chunk;
    }
    return false;
}
#endif

__device__ __forceinline__ float combine(float a, float b, unsigned int red_op) {
    if (red_op == 0) return __fadd_rn(a, b);
    if (red_op == 1) return (b < a) ? b : a;
    return (a < b) ? b : a;
}

// ---- staging.  Every load step of a task is brought from global memory to shared memory with
// cp.async (16 bytes per instruction, L2 only), several steps ahead of its use.  A thread only ever
// reads back the bytes it copied itself, so no barrier is needed: cp.async.wait_group orders them.
// Shared layout of one stage: [vector j][thread] of 16-byte vectors (conflict free).
//   F32 task:  vector j (of 4) of thread t holds elements (j*256 + t)*4 .. +3 of the tile.
//   BF16 task: group j (of 2) of thread t holds elements (j*256 + t)*8 .. +7: one vector for a bf16
//              operand, two (slots 2j, 2j+1) for an fp32 operand (a materialised partial result).
// Stage count per kernel variant: with up to 4 accumulators two CTAs share an SM (6 stages each, 5 steps =
// 40-80 KiB per CTA in flight); the 8-accumulator variant needs the whole register file of an SM for one
// CTA and gets 12 stages instead.
constexpr int kStageBytes = 4 * kReduceThreads * 16;
constexpr int kVecStride = kReduceThreads * 16;   // bytes between a thread's consecutive vectors, in shared and (mostly) global
// A variant that also fans its result out (FAN) keeps one more 16 KiB buffer for the result tile, from which the
// bulk copies read, and gives up one stage for it where two CTAs share an SM.
template <int A, bool FAN = false>
struct StagesFor {
    static constexpr int value = A <= 4 ? (FAN ? 5 : 6) : 12;
    static constexpr int min_ctas = A <= 4 ? 2 : 1;
    static constexpr int smem_bytes = value * kStageBytes + (FAN ? kStageBytes : 0);
};

// A step as the kernel keeps it in shared memory: the packed record of the wave (operand address in the low
// 56 bits; code, accumulator and operand kind on top).  A load step whose address is 0 is resolved through the
// device directory (the row beside it) when the task's records are set up.
__device__ __forceinline__ unsigned int rec_meta(unsigned long long rec) { return (unsigned int)(rec >> kRecShift); }
__device__ __forceinline__ unsigned int meta_code(unsigned int m) { return m & 3u; }
__device__ __forceinline__ unsigned int meta_acc(unsigned int m) { return (m >> 2) & 7u; }
__device__ __forceinline__ bool meta_is_bf16(unsigned int m) { return (m & 32u) != 0; }

__device__ __forceinline__ void cp_async16_partial(unsigned int smem_addr, unsigned long long gaddr, unsigned int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_addr), "l"(gaddr), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ unsigned long long ld_shared_u64(unsigned int addr) {
    unsigned long long v;
    asm volatile("ld.shared.u64 %0, [%1];" : "=l"(v) : "r"(addr));
    return v;
}

// Sixteen fp32 values of a thread as eight register pairs, so that sums can use the packed fp32 add of
// sm_100 (two IEEE round-to-nearest adds per instruction; same bits as two scalar adds).
struct Acc {
    unsigned long long p[8];
};
__device__ __forceinline__ unsigned long long pack2(unsigned int lo, unsigned int hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, unsigned int& lo, unsigned int& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
    unsigned long long r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ void combine_acc(Acc& a, const Acc& x, unsigned int red_op) {
    if (red_op == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) a.p[i] = add2(a.p[i], x.p[i]);
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            unsigned int al, ah, xl, xh;
            unpack2(a.p[i], al, ah);
            unpack2(x.p[i], xl, xh);
            const float l = combine(__uint_as_float(al), __uint_as_float(xl), red_op);
            const float h = combine(__uint_as_float(ah), __uint_as_float(xh), red_op);
            a.p[i] = pack2(__float_as_uint(l), __float_as_uint(h));
        }
    }
}

template <bool BF16, int kStages>
struct TileCtx {
    unsigned int rec_base;             // shared-window address of the step records
    unsigned int n, pc, red_op;
    unsigned int issue_idx;            // next step whose copy is to be started
    unsigned int issue_stage, cons_stage, stage_lo, stage_end;   // this thread's slot in the stage ring
    unsigned long long goff_main;      // byte offset of this thread's first vector for the wave's source dtype
    unsigned long long goff_f32;       // (BF16 waves) the same for an fp32 operand
    unsigned int count, t;             // elements in the tile, thread index
    unsigned int nb_main[BF16 ? 2 : 4];  // bytes of each of this thread's vectors that lie inside the tile (16 unless ragged)

    // bytes of a 16-byte vector starting at element `off` of the tile that lie inside it
    __device__ __forceinline__ unsigned int inside(unsigned int off, unsigned int per_vec, unsigned int elem_bytes) const {
        const unsigned int left = off < count ? count - off : 0u;
        return (left < per_vec ? left : per_vec) * elem_bytes;
    }

    __device__ __forceinline__ void advance(unsigned int& stage) {
        stage += kStageBytes;
        if (stage == stage_end) stage = stage_lo;
    }

    __device__ __forceinline__ void issue() {
        if (issue_idx < n) {
            const unsigned long long rec = ld_shared_u64(rec_base + issue_idx * 8);
            const unsigned int m = rec_meta(rec);
            if (meta_code(m) != OPC_ADD_ACC) {
                const unsigned long long ptr = rec & ((1ull << kRecShift) - 1);
                if (!BF16 || meta_is_bf16(m)) {
                    const unsigned long long g = ptr + goff_main;
#pragma unroll
                    for (int j = 0; j < (BF16 ? 2 : 4); ++j) {
                        // a vector that lies (partly) beyond the tile copies fewer bytes, or none, and is zero-filled
                        cp_async16_partial(issue_stage + j * kVecStride, g + j * kVecStride, nb_main[j]);
                    }
                } else {
                    const unsigned long long g = ptr + goff_f32;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const unsigned int go = (j >> 1) * (2 * kVecStride) + (j & 1) * 16;
                        const unsigned int nb = inside(((j >> 1) * kReduceThreads + t) * 8 + (j & 1) * 4, 4, 4);
                        cp_async16_partial(issue_stage + j * kVecStride, g + go, nb);
                    }
                }
            }
        }
        cp_async_commit();  // one group per step, empty or not, keeps the group count equal to the step count
        ++issue_idx;
        advance(issue_stage);
    }

    // Consumes step pc: starts the copy kStages-1 steps ahead, waits for this step's bytes, widens to fp32.
    __device__ __forceinline__ void fetch(unsigned int m, Acc& x) {
        issue();
        cp_async_wait<kStages - 1>();
        uint4 v[4];
        const bool half = BF16 && meta_is_bf16(m);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (j < 2 || !BF16 || !half) {
                const unsigned int a = cons_stage + j * kVecStride;
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v[j].x), "=r"(v[j].y), "=r"(v[j].z), "=r"(v[j].w) : "r"(a));
            }
        }
        if (!half) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                x.p[j * 2 + 0] = pack2(v[j].x, v[j].y);
                x.p[j * 2 + 1] = pack2(v[j].z, v[j].w);
            }
        } else {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const unsigned int w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
                for (int i = 0; i < 4; ++i) x.p[j * 4 + i] = pack2(w[i] << 16, w[i] & 0xFFFF0000u);  // bf16 -> fp32 is exact
            }
        }
        advance(cons_stage);
        ++pc;
    }

    __device__ __forceinline__ void skip() {  // an ADD_ACC step: no bytes, but its (empty) group is counted
        issue();
        advance(cons_stage);
        ++pc;
    }
};

// Runs the steps that belong to accumulator L, starting at a LOAD into L, until a step that belongs to
// a shallower accumulator.  A step into L+1 opens a fused child subtree: one more level of this
// function, whose accumulator is a separate set of registers, closed by ADD_ACC(L, L+1).
template <int L, int A, bool BF16, bool FAN>
__device__ __forceinline__ void eval_level(TileCtx<BF16, StagesFor<A, FAN>::value>& cx, Acc& acc) {
    while (cx.pc < cx.n) {
        const unsigned int m = rec_meta(ld_shared_u64(cx.rec_base + cx.pc * 8));
        const unsigned int a = meta_acc(m);
        if (L > 0 && (int)a < L) return;
        if ((int)a == L) {
            Acc x;
            cx.fetch(m, x);
            if (meta_code(m) == OPC_LOAD) {
#pragma unroll
                for (int i = 0; i < 8; ++i) acc.p[i] = x.p[i];
            } else {
                combine_acc(acc, x, cx.red_op);
            }
        } else {
            if constexpr (L + 1 < A) {
                Acc sub;
                eval_level<L + 1, A, BF16, FAN>(cx, sub);
                cx.skip();  // the ADD_ACC(L, L+1) that closes the subtree
                combine_acc(acc, sub, cx.red_op);
            } else {
                cx.skip();  // unreachable for a well-formed task (the planner bounds the depth by A)
            }
        }
    }
}

constexpr int kFanIssuers = 64;   // threads that issue the bulk copies of a fused fan-out

__device__ __forceinline__ void bulk_store(unsigned long long gdst, unsigned int smem_src, unsigned int bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_src), "r"(bytes) : "memory");
}

template <int A, bool BF16, bool FAN>
__device__ __forceinline__ void run_tile(unsigned int rec_base, unsigned int stage_base, const ReduceTask& task, unsigned long long e0,
                                         unsigned int count, unsigned int t, const unsigned long long* fan_ptrs) {
    constexpr int kStages = StagesFor<A, FAN>::value;
    TileCtx<BF16, kStages> cx;
    cx.rec_base = rec_base;
    cx.n = task.n_steps;
    cx.pc = 0;
    cx.red_op = task.red_op;
    cx.issue_idx = 0;
    cx.stage_lo = stage_base + t * 16;
    cx.stage_end = cx.stage_lo + kStages * kStageBytes;
    cx.issue_stage = cx.cons_stage = cx.stage_lo;
    if (!BF16) {
        cx.goff_main = e0 * 4ull + t * 16ull;
        cx.goff_f32 = cx.goff_main;
    } else {
        cx.goff_main = e0 * 2ull + t * 16ull;
        cx.goff_f32 = e0 * 4ull + t * 32ull;
    }
    cx.count = count;
    cx.t = t;
#pragma unroll
    for (int j = 0; j < (BF16 ? 2 : 4); ++j)
        cx.nb_main[j] = BF16 ? cx.inside((j * kReduceThreads + t) * 8, 8, 2) : cx.inside((j * kReduceThreads + t) * 4, 4, 4);
#pragma unroll
    for (int i = 0; i < kStages - 1; ++i) cx.issue();

    Acc acc;
    eval_level<0, A, BF16, FAN>(cx, acc);
    cp_async_wait<0>();

    float* out = reinterpret_cast<float*>(task.out_ptr) + e0;
    if constexpr (FAN) {
        if (task.n_fan != 0) {
            // Fused fan-out (reduce followed by broadcast, Section 3.4.3): the result tile goes registers -> shared
            // memory -> one bulk copy to the target and one to every receiver.  The tile's whole 16-byte vectors
            // travel by bulk copy, the last elements of an object whose length is not a multiple of 4 by plain stores.
            const unsigned int s_out = stage_base + kStages * kStageBytes;
            if (t < kFanIssuers) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the previous tile's copies have read the buffer
            __syncthreads();
            const unsigned int n_vec_bytes = (count / 4u) * 16u;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const unsigned int off = BF16 ? ((q >> 1) * kReduceThreads + t) * 8 + (q & 1) * 4 : (q * kReduceThreads + t) * 4;
                unsigned int r[4];
                unpack2(acc.p[q * 2 + 0], r[0], r[1]);
                unpack2(acc.p[q * 2 + 1], r[2], r[3]);
                asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(s_out + off * 4u), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
                if (off < count && off + 4 > count) {     // the ragged last vector: element by element, to every destination
                    for (unsigned int d = 0; d <= task.n_fan; ++d) {
                        float* o = d == 0 ? out : reinterpret_cast<float*>(fan_ptrs[task.fan_begin + d - 1]) + e0;
                        for (int i = 0; i < 4; ++i)
                            if (off + i < count) o[off + i] = __uint_as_float(r[i]);
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // make the tile visible to the bulk-copy engine
            __syncthreads();
            if (t < kFanIssuers) {
                if (n_vec_bytes != 0) {
                    for (unsigned int d = t; d <= task.n_fan; d += kFanIssuers) {
                        const unsigned long long base = d == 0 ? task.out_ptr : fan_ptrs[task.fan_begin + d - 1];
                        bulk_store(base + e0 * 4ull, s_out, n_vec_bytes);
                    }
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
            return;
        }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const unsigned int off = BF16 ? ((q >> 1) * kReduceThreads + t) * 8 + (q & 1) * 4 : (q * kReduceThreads + t) * 4;
        unsigned int r[4];
        unpack2(acc.p[q * 2 + 0], r[0], r[1]);
        unpack2(acc.p[q * 2 + 1], r[2], r[3]);
        if (off + 4 <= count) {
            *reinterpret_cast<uint4*>(out + off) = make_uint4(r[0], r[1], r[2], r[3]);
        } else {
            for (int i = 0; i < 4; ++i)
                if (off + i < count) out[off + i] = __uint_as_float(r[i]);
        }
    }
}

template <int A, bool BF16, bool FAN>
__global__ void __launch_bounds__(kReduceThreads, StagesFor<A, FAN>::min_ctas) reduce_wave_kernel(const __grid_constant__ ReduceWave w) {
    extern __shared__ __align__(16) unsigned char s_stage[];
    __shared__ unsigned long long s_rec[kMaxStepsPerWave];
    const unsigned int t = threadIdx.x;
    const unsigned long long t_start = global_timer_ns();
    const unsigned int rec_base = (unsigned int)__cvta_generic_to_shared(s_rec);
    const unsigned int stage_base = (unsigned int)__cvta_generic_to_shared(s_stage);
    int cached_task = -1;

    for (unsigned int g = blockIdx.x; g < w.total_tiles; g += gridDim.x) {
        int ti = 0;
        while (ti + 1 < (int)w.n_tasks && g >= w.tasks[ti + 1].tile_begin) ++ti;
        const ReduceTask& task = w.tasks[ti];
        if (ti != cached_task) {
            __syncthreads();  // everyone is done with the previous task's records
            for (unsigned int i = t; i < task.n_steps; i += kReduceThreads) {
                unsigned long long rec = w.recs[task.step_begin + i];
                if (meta_code(rec_meta(rec)) != OPC_ADD_ACC && (rec & ((1ull << kRecShift) - 1)) == 0ull)
                    rec |= w.dir[w.rows[task.step_begin + i]].ptr & ((1ull << kRecShift) - 1);
                s_rec[i] = rec;
            }
            cached_task = ti;
            __syncthreads();
        }
        const unsigned int lt = g - task.tile_begin;
        const unsigned int c = task.c_begin + lt / task.tiles_per_chunk;
        const unsigned int j = lt % task.tiles_per_chunk;
        const unsigned long long e0 = (unsigned long long)c * task.chunk_elems + (unsigned long long)j * kTileElems;
        unsigned long long e1 = e0 + kTileElems;
        const unsigned long long chunk_end = (unsigned long long)(c + 1) * task.chunk_elems;
        if (e1 > chunk_end) e1 = chunk_end;
        if (e1 > task.elems) e1 = task.elems;
        if (e0 >= e1) continue;

        if (task.poll) {
            int ok = 1;
            for (unsigned int i = t; i < task.n_steps; i += kReduceThreads) {
                if (meta_code(rec_meta(w.recs[task.step_begin + i])) != OPC_ADD_ACC)
                    ok &= wait_chunk(w.dir, w.status, w.rows[task.step_begin + i], c, t_start, w.budget_ns) ? 1 : 0;
            }
            if (!__syncthreads_and(ok)) break;
        }

        const unsigned int count = (unsigned int)(e1 - e0);
#ifdef HPL_DEBUG_BOUNDS
        if (task.out_row != 0xFFFFFFFFu) {   // (a task without directory rows of its own is not checked)
            int ok = 1;
            for (unsigned int i = t; i < task.n_steps; i += kReduceThreads) {
                const unsigned long long rec = w.recs[task.step_begin + i];
                const unsigned int m = rec_meta(rec);
                if (meta_code(m) == OPC_ADD_ACC) continue;
                const unsigned long long es = (BF16 && meta_is_bf16(m)) ? 2ull : 4ull;
                ok &= range_ok(w.dir, w.status, w.rows[task.step_begin + i], s_rec[i], e0 * es, e1 * es, c) ? 1 : 0;
            }
            if (t == 0) ok &= range_ok(w.dir, w.status, task.out_row, task.out_ptr, e0 * 4ull, e1 * 4ull, c) ? 1 : 0;
            for (unsigned int i = t; i < task.n_fan; i += kReduceThreads)
                ok &= range_ok(w.dir, w.status, w.fan_rows[task.fan_begin + i], w.fan_ptrs[task.fan_begin + i], e0 * 4ull, e1 * 4ull, c) ? 1 : 0;
            if (!__syncthreads_and(ok)) continue;
        }
#endif
        run_tile<A, BF16, FAN>(rec_base, stage_base, task, e0, count, t, w.fan_ptrs);
    }
    if constexpr (FAN) {
        // shared memory must stay valid until the bulk copies have read it, and their writes must be complete
        if (t < kFanIssuers) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
}

// ------------------------------------------------------------------------------------------ fan-out
// A tile is loaded once (16-byte loads, L2 only) into one of two shared-memory buffers and then written to
// every receiver with one bulk copy per receiver (shared -> global, cp.async.bulk, issued by the first 64
// threads): large contiguous writes reach a higher HBM write rate than per-thread stores, and the next
// tile's load overlaps the draining stores.  The only waits are on the CTA's own bulk copies
// (cp.async.bulk.wait_group), which always complete.
constexpr int kFanoutIssuers = 64;
constexpr int kFanoutSmemBytes = 2 * kFanoutTileBytes;

__global__ void __launch_bounds__(kFanoutThreads) fanout_wave_kernel(const __grid_constant__ FanoutWave w) {
    extern __shared__ __align__(128) unsigned char s_tile[];
    __shared__ unsigned long long s_dst[kMaxFanoutDst];
    __shared__ unsigned long long s_src;
    const unsigned int t = threadIdx.x;
    const unsigned long long t_start = global_timer_ns();
    int cached_task = -1;
    unsigned int buf = 0;

    for (unsigned int g = blockIdx.x; g < w.total_tiles; g += gridDim.x) {
        int ti = 0;
        while (ti + 1 < (int)w.n_tasks && g >= w.tasks[ti + 1].tile_begin) ++ti;
        const FanoutTask& task = w.tasks[ti];
        if (ti != cached_task) {
            __syncthreads();
            for (unsigned int i = t; i < task.n_dst; i += kFanoutThreads) s_dst[i] = w.dst_ptrs[task.dst_begin + i];
            if (t == 0) s_src = task.src_ptr;
            cached_task = ti;
            __syncthreads();
        }
        const unsigned int lt = g - task.tile_begin;
        const unsigned int c = task.c_begin + lt / task.tiles_per_chunk;
        const unsigned int j = lt % task.tiles_per_chunk;
        const unsigned long long b0 = (unsigned long long)c * task.chunk_bytes + (unsigned long long)j * task.tile_bytes;
        unsigned long long b1 = b0 + task.tile_bytes;
        const unsigned long long chunk_end = (unsigned long long)(c + 1) * task.chunk_bytes;
        if (b1 > chunk_end) b1 = chunk_end;
        if (b1 > task.bytes) b1 = task.bytes;
        if (b0 >= b1) continue;

        if (task.poll) {
            int ok = 1;
            if (t == 0) ok = wait_chunk(w.dir, w.status, task.src_row, c, t_start, w.budget_ns) ? 1 : 0;
            if (!__syncthreads_and(ok)) break;
        }

#ifdef HPL_DEBUG_BOUNDS
        {
            int ok = 1;
            if (t == 0) ok = range_ok(w.dir, w.status, task.src_row, task.src_ptr, b0, b1, c) ? 1 : 0;
            for (unsigned int i = t; i < task.n_dst; i += kFanoutThreads)
                ok &= range_ok(w.dir, w.status, w.dst_rows[task.dst_begin + i], w.dst_ptrs[task.dst_begin + i], b0, b1, c) ? 1 : 0;
            if (!__syncthreads_and(ok)) continue;
        }
#endif
        // the bulk copies that read this buffer two tiles ago must have finished reading it
        if (t < kFanoutIssuers) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        __syncthreads();

        unsigned char* tile = s_tile + buf * kFanoutTileBytes;
        const unsigned char* src = reinterpret_cast<const unsigned char*>(s_src) + b0;
        const unsigned int count = (unsigned int)(b1 - b0);
        const unsigned int n_vec = count / 16;
        constexpr int kVecPerThread = kFanoutTileBytes / 16 / kFanoutThreads;
        uint4 v[kVecPerThread];
#pragma unroll
        for (int q = 0; q < kVecPerThread; ++q) {
            const unsigned int i = q * kFanoutThreads + t;
            if (i < n_vec) v[q] = __ldcg(reinterpret_cast<const uint4*>(src) + i);
        }
#pragma unroll
        for (int q = 0; q < kVecPerThread; ++q) {
            const unsigned int i = q * kFanoutThreads + t;
            if (i < n_vec) reinterpret_cast<uint4*>(tile)[i] = v[q];
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // make the tile visible to the bulk-copy engine
        __syncthreads();
        const unsigned int n_dst = task.n_dst;
        if (t < kFanoutIssuers) {
            if (n_vec) {
                const unsigned int sa = (unsigned int)__cvta_generic_to_shared(tile);
                for (unsigned int r = t; r < n_dst; r += kFanoutIssuers) bulk_store(s_dst[r] + b0, sa, n_vec * 16);
            }
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        // the last bytes of an object whose size is not a multiple of 16
        for (unsigned int b = n_vec * 16 + t; b < count; b += kFanoutThreads) {
            const unsigned char x = src[b];
            for (unsigned int r = 0; r < n_dst; ++r) (reinterpret_cast<unsigned char*>(s_dst[r]) + b0)[b] = x;
        }
        buf ^= 1u;
    }
    // shared memory must stay valid until the bulk copies have read it, and the writes must be complete
    if (t < kFanoutIssuers) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// ------------------------------------------------------------------------------------------ launchers
// Per device and kernel variant: the dynamic shared memory attribute is set and the occupancy asked for once,
// under a lock (cudaFuncSetAttribute is per device; contexts and hpl_reduce_noalloc may run on several threads).
namespace {

constexpr int kVariants = 13;   // 3 accumulator classes x {f32, bf16} x {plain, fan} reduce variants + the fan-out kernel
std::mutex g_variant_mu;
std::vector<std::array<int, kVariants>> g_occ_of_device;   // 0 = not prepared yet

int variant_index(int n_acc, bool bf16, bool fan) { return ((n_acc <= 2 ? 0 : (n_acc <= 4 ? 1 : 2)) * 2 + (bf16 ? 1 : 0)) * 2 + (fan ? 1 : 0); }

template <int A, bool BF16, bool FAN>
int prepare_reduce_variant() {
    int n = 0;
    if (cudaFuncSetAttribute(reduce_wave_kernel<A, BF16, FAN>, cudaFuncAttributeMaxDynamicSharedMemorySize, StagesFor<A, FAN>::smem_bytes) != cudaSuccess) return -1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, reduce_wave_kernel<A, BF16, FAN>, kReduceThreads, StagesFor<A, FAN>::smem_bytes) != cudaSuccess) return -1;
    return n < 1 ? 1 : n;
}

template <int A>
int prepare_reduce_a(bool bf16, bool fan) {
    if (bf16) return fan ? prepare_reduce_variant<A, true, true>() : prepare_reduce_variant<A, true, false>();
    return fan ? prepare_reduce_variant<A, false, true>() : prepare_reduce_variant<A, false, false>();
}

int prepare_fanout() {
    int n = 0;
    if (cudaFuncSetAttribute(fanout_wave_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFanoutSmemBytes) != cudaSuccess) return -1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fanout_wave_kernel, kFanoutThreads, kFanoutSmemBytes) != cudaSuccess) return -1;
    if (n > 2) n = 2;   // two CTAs per SM already saturate the write path
    return n < 1 ? 1 : n;
}

// CTAs per SM of a variant on the current device (prepares it at first use); -1 on a CUDA error.
int variant_occupancy(int idx, int n_acc, bool bf16, bool fan) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    std::lock_guard<std::mutex> lock(g_variant_mu);
    if ((int)g_occ_of_device.size() <= dev) g_occ_of_device.resize(dev + 1, std::array<int, kVariants>{});
    int& occ = g_occ_of_device[dev][idx];
    if (occ == 0) {
        int n;
        if (idx == kVariants - 1) n = prepare_fanout();
        else if (n_acc <= 2) n = prepare_reduce_a<2>(bf16, fan);
        else if (n_acc <= 4) n = prepare_reduce_a<4>(bf16, fan);
        else n = prepare_reduce_a<kMaxAcc>(bf16, fan);
        if (n < 0) return -1;
        occ = n;
    }
    return occ;
}

template <int A, bool BF16, bool FAN>
int launch_reduce_t(const ReduceWave& w, int grid, cudaStream_t s) {
    reduce_wave_kernel<A, BF16, FAN><<<grid, kReduceThreads, StagesFor<A, FAN>::smem_bytes, s>>>(w);
    return (int)cudaGetLastError();
}

template <int A>
int launch_reduce_a(const ReduceWave& w, bool bf16, bool fan, int grid, cudaStream_t s) {
    if (bf16) return fan ? launch_reduce_t<A, true, true>(w, grid, s) : launch_reduce_t<A, true, false>(w, grid, s);
    return fan ? launch_reduce_t<A, false, true>(w, grid, s) : launch_reduce_t<A, false, false>(w, grid, s);
}

}  // namespace

int reduce_ctas_per_sm(int n_acc, bool bf16, bool fan) {
    const int n = variant_occupancy(variant_index(n_acc, bf16, fan), n_acc, bf16, fan);
    return n < 1 ? 1 : n;
}

int fanout_ctas_per_sm() {
    const int n = variant_occupancy(kVariants - 1, 0, false, false);
    return n < 1 ? 1 : n;
}

int launch_reduce_wave(const ReduceWave& w, int n_acc, bool bf16, bool fan, int grid, void* stream) {
    cudaStream_t s = (cudaStream_t)stream;
    if (variant_occupancy(variant_index(n_acc, bf16, fan), n_acc, bf16, fan) < 0) return (int)cudaErrorUnknown;
    if (n_acc <= 2) return launch_reduce_a<2>(w, bf16, fan, grid, s);
    if (n_acc <= 4) return launch_reduce_a<4>(w, bf16, fan, grid, s);
    return launch_reduce_a<kMaxAcc>(w, bf16, fan, grid, s);
}

int launch_fanout_wave(const FanoutWave& w, int grid, void* stream) {
    if (variant_occupancy(kVariants - 1, 0, false, false) < 0) return (int)cudaErrorUnknown;
    fanout_wave_kernel<<<grid, kFanoutThreads, kFanoutSmemBytes, (cudaStream_t)stream>>>(w);
    return (int)cudaGetLastError();
}

}  // namespace hpl
